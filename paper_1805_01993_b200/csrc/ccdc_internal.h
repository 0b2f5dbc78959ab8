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
#ifndef CCDC_DECODE_FILES_MAX
#define CCDC_DECODE_FILES_MAX 4         // most files of a batch loaded together (4, 2; 1 = batch-by-batch kernel)
#endif
#ifndef CCDC_DECODE_GROUP_WORDS
#define CCDC_DECODE_GROUP_WORDS 40      // most words per thread a batch may keep in flight
#endif
#ifndef CCDC_DECODE_VECTORS
#define CCDC_DECODE_VECTORS 1       // vectors per thread per tile
#endif
#ifndef CCDC_DECODE_DEPTH
#define CCDC_DECODE_DEPTH 2         // batches whose loads are issued together (one-file batches, r <= 4)
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
    int device = -1;          // device holding the table copies, -1 = none
    void *d_blob = nullptr;   // one allocation for all of them
};

// implemented in ccdc_plan.cpp: sizes the split of the fused decode again for a device with sm_count SMs
void ccdc_internal_resplit(ccdc_plan_s *plan, int sm_count);
// implemented in ccdc_kernels.cu
void ccdc_internal_release_device(ccdc_plan_s *plan);
int ccdc_internal_cuda_fail(int cuda_error);    // records the error for ccdc_last_cuda_error; returns CCDC_ECUDA
void ccdc_internal_count_launch();              // one more kernel launched by the library
