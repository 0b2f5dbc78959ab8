// Internal plan representation shared by the host planner and the launch code.
#pragma once

#include <cstdint>
#include <vector>

#include "ccdc.h"

// Launch shapes (build-time options).  The fused decode+reduce keeps its loads
// in registers; the gather kernel streams through a shared-memory pipeline.
// The planner sizes the split of the fused decode from the decode tile.
#ifndef CCDC_DECODE_THREADS
#define CCDC_DECODE_THREADS 512     // threads per block
#endif
#ifndef CCDC_DECODE_THREADS_SHORT
#define CCDC_DECODE_THREADS_SHORT 1024  // used instead when one such block covers a whole segment
#endif
#ifndef CCDC_DECODE_THREADS_FILES
#define CCDC_DECODE_THREADS_FILES 128   // used when several files of a batch are loaded together
#endif
#ifndef CCDC_DECODE_BLOCKS_FILES         // blocks of that kernel resident per SM, by vector width (planner and kernel agree)
#define CCDC_DECODE_BLOCKS_FILES(vec) ((vec) <= 2 ? 7 : 6)
#endif
#ifndef CCDC_DECODE_FILES_MAX
#define CCDC_DECODE_FILES_MAX 4         // most files of a batch loaded together (4, 2; 1 = batch-by-batch kernel)
#endif
#ifndef CCDC_DECODE_GROUP_WORDS
#define CCDC_DECODE_GROUP_WORDS 40      // most words per thread a batch may keep in flight
#endif
#ifndef CCDC_STREAM_TILE_WORDS
#define CCDC_STREAM_TILE_WORDS 2048     // bulk-copy pipeline: words of a segment per block (a multiple of 512)
#endif
#ifndef CCDC_STREAM_SMEM_BYTES
#define CCDC_STREAM_SMEM_BYTES (72 * 1024)  // bulk-copy pipeline: shared memory per block (three blocks per SM)
#endif
#ifndef CCDC_DECODE_CLUSTER_SUM
#define CCDC_DECODE_CLUSTER_SUM 1       // split batch loop of up to 8 chunks (several files per batch): sum through a cluster
#endif
#ifndef CCDC_DECODE_VECTORS
#define CCDC_DECODE_VECTORS 1       // vectors per thread per tile
#endif
#ifndef CCDC_DECODE_DEPTH
#define CCDC_DECODE_DEPTH 2         // batches whose loads are issued together (one-file batches, r <= 4)
#endif
#ifndef CCDC_DECODE_DEPTH_FILES
#define CCDC_DECODE_DEPTH_FILES 3   // the same when several files of a batch are loaded together
#endif
#ifndef CCDC_DECODE_DEPTH_WORDS
#define CCDC_DECODE_DEPTH_WORDS 20  // a batch of more words per thread than this is not overlapped with the next
#endif
#ifndef CCDC_GATHER_THREADS
#define CCDC_GATHER_THREADS 128
#endif
#ifndef CCDC_GATHER_VECTORS
#define CCDC_GATHER_VECTORS 4       // vectors per thread per chunk
#endif
#ifndef CCDC_GATHER_STAGES
#define CCDC_GATHER_STAGES 4        // chunks in flight per thread
#endif

// One operand of a gathered segment: element offset into the owning node's
// buffer (segment offset included) and the number of leading elements of the
// segment that exist (the rest is the virtual zero extension).
struct ccdc_ref {
    long long off;
    long long vl;
};

// One destination row of the gather kernel:
//   dst[dst_node][dst_off + j] = coded_in[coded_off + j] (if coded_off >= 0)
//                                XOR_a  [j < vl_a] * sum_f src[src_node][off_a + f*file_stride + j]
// for j < n.
struct ccdc_row {
    int src_node;
    int dst_node;
    long long dst_off;
    long long n;
    long long coded_off;
    long long nf;           // files summed per operand; 0 = the plan's files per batch
};

// A table of gather rows with a fixed number of operands per row.
struct ccdc_gather_table {
    std::vector<ccdc_row> rows;
    std::vector<ccdc_ref> refs;     // [rows][na]
    int na = 0;
    long long n_max = 0;            // largest row length
    bool uniform = true;            // no row carries its own file count (nf = 0 everywhere)
    long long nf_max = 0;           // largest per-row file count (tables that are not uniform)
    // device copies
    const ccdc_row *d_rows = nullptr;
    const ccdc_ref *d_refs = nullptr;
};

// Bulk-copy pipeline (ccdc_stream.cu): the source rows of an output segment
// (decode) or of a coded row (encode), flattened.  A "cell" is one output
// segment / coded row; its rows are listed in the order they are folded.
enum {
    CCDC_SROW_FIRST_FILE = 1,   // first file of an operand: starts the file sum
    CCDC_SROW_LAST_FILE = 2,    // last file of an operand: the sum enters the batch's XOR
    CCDC_SROW_CODED = 4,        // a coded packet: starts the batch's XOR as it is
    CCDC_SROW_FIRST_OP = 8,     // first operand of a batch
    CCDC_SROW_LAST_OP = 16,     // last operand of a batch: the XOR is added to the output
    CCDC_SROW_FROM_CODED = 32   // the row is read from the coded buffer, not from the node's partition
};
struct ccdc_stream_row {
    long long off;      // word offset of the segment in its buffer
    int vl;             // leading words of the segment that exist
    int flags;
};
struct ccdc_stream_cell {
    long long row0;     // first entry of the cell in the row list
    long long dst_off;  // word offset of the cell's output
    int src_node;       // whose partition the rows are read from
    int seglen;         // words of the output
};
struct ccdc_stream_table {
    std::vector<ccdc_stream_row> rows;
    std::vector<ccdc_stream_cell> cells;
    std::vector<int> chunk_row0;        // [cells][nchunk + 1]: first row of each chunk of the batch loop, cell relative
    const ccdc_stream_row *d_rows = nullptr;
    const ccdc_stream_cell *d_cells = nullptr;
    const int *d_chunk_row0 = nullptr;
};

struct ccdc_plan_s {
    int K = 0, r = 0, Q = 0, dtype = 0;
    bool jobs_mode = false;
    bool compression_mode = false;  // the appendix's compression-only comparator (no coding)
    std::vector<long long> node_nfiles;     // [K] files stored at node k
    // node-sharded plans (several GPUs, K/world nodes each): this rank's share
    int shard_rank = 0, shard_world = 1;
    long long send_rows = 0;                // coded rows this rank encodes (= every rank's)
    std::vector<long long> coded_row_pos;   // [nround*(r+1)] position of a coded row in the gathered buffer
    std::vector<int> out_rows;              // out rows (job*K + node) of this rank's nodes, ascending
    const int *d_out_rows = nullptr;
    long long N = 0, B = 0, J = 1;
    long long b = 0;          // files per batch
    long long len = 0;        // (Q/K)*B
    long long s = 0;          // ceil(len/r)
    long long s_pad = 0;      // coded row stride (multiple of 4 words)
    long long row_elems = 0;  // Q*B: elements of one file at a node
    long long nbatch = 0, nround = 0, nterm = 0;   // nterm = batches per job
    int vec = 1;              // widest vector (words) dividing s and len: 4, 2 or 1
    int term_stride = 0;      // refs per term of the fused decode: 1 + max(r-1, 1)
    int decode_threads = CCDC_DECODE_THREADS;   // block size of the fused decode
    int decode_files = 1;     // files of a batch whose loads the fused decode issues together
    bool decode_cluster = false;    // the chunks of an output tile meet in a thread-block cluster (no workspace)
    bool tuned = false;       // the caller fixed the decode's launch shape (ccdc_plan_tune_decode)
    int nchunk = 1;           // split of the batch loop in the fused decode
    long long terms_per_chunk = 0;

    std::vector<int> batch_nodes;           // [nbatch][r]
    std::vector<long long> batch_file0;     // [nbatch]
    std::vector<long long> batch_job;       // [nbatch]
    std::vector<long long> job_batch0;      // [J] first batch id of job j (a job's batches are consecutive)
    std::vector<int> round_group;           // [nround][r+1]
    std::vector<long long> round_batch;     // [nround][r+1]
    std::vector<long long> slot;            // [K][nbatch] local index or -1
    std::vector<long long> nlocal;          // [K]
    std::vector<long long> recv_round;      // [nbatch][K]
    std::vector<long long> node_round_index;// [nround][r+1]: index of the round among member a's rounds
    std::vector<long long> node_nrounds;    // [K]

    // gather tables: fused encode (from partitions), and the stepwise
    // combine / encode / decode (through materialised packets)
    ccdc_gather_table enc_fused, cmb, enc_pk, dec_pk;
    // fused decode+reduce: [out rows][r][nterm][term_stride]
    //   ref 0: {coded offset, s} or {-1, 0} for a batch stored locally
    //   ref 1..: partition rows to cancel (or, locally, the row to add)
    std::vector<ccdc_ref> dec_terms;
    const ccdc_ref *d_dec_terms = nullptr;
    // stepwise reduce: [out rows][nterm]: vl = 0 partition row (sum of b files), vl = 1 decoded row
    std::vector<ccdc_ref> red_terms;
    const ccdc_ref *d_red_terms = nullptr;

    int sm_count = 148;       // SMs the launch shapes are sized for (the device's count once uploaded)
    int family = 0;           // 0: loads through registers; 1: bulk-copy pipelines (ccdc_stream.cu)
    bool family_tuned = false;
    int device_has_bulk_copies = 1;     // compute capability >= 9.0 (known once uploaded)
    int *d_status = nullptr;  // one word, set by a kernel whose bounded wait ran out
    ccdc_stream_table enc_stream, dec_stream;   // built at upload for family 1
    int device = -1;          // device holding the table copies, -1 = none
    void *d_blob = nullptr;   // one allocation for all of them
};

// implemented in ccdc_plan.cpp: sizes the split of the fused decode again for a device with sm_count SMs
void ccdc_internal_resplit(ccdc_plan_s *plan, int sm_count);
// implemented in ccdc_plan.cpp: the row lists of the bulk-copy pipeline for the plan's final split
void ccdc_internal_build_stream_tables(ccdc_plan_s *plan);
// implemented in ccdc_plan.cpp: the split for the plan's current kernel family
void ccdc_internal_choose_split(ccdc_plan_s *plan);
// implemented in ccdc_kernels.cu
void ccdc_internal_release_device(ccdc_plan_s *plan);
int ccdc_internal_cuda_fail(int cuda_error);    // records the error for ccdc_last_cuda_error; returns CCDC_ECUDA
void ccdc_internal_count_launch();              // one more kernel launched by the library
