/*
 * ccdc.h -- C ABI of the compressed coded distributed computing (compressed
 * CDC) shuffle for one NVIDIA B200 (sm_100a).
 *
 * The method is that of Li, Maddah-Ali and Avestimehr, "Compressed Coded
 * Distributed Computing": a MapReduce job with linear aggregation (Eq. (1)),
 * N files placed on K nodes with computation load r = mu*K (Section IV-A),
 * Q Reduce functions, Q/K per node (Section III).  In the Shuffle phase every
 * node pre-combines, by summation over a batch of files, the intermediate
 * values another node needs, XORs equal segments of r such packets into one
 * coded multicast packet per (r+1)-subset, and every receiver cancels what it
 * can rebuild from its own Map results (Section IV-B).
 *
 * Here the K nodes are logical: each node's Map results live in a partition of
 * one GPU's memory, and a multicast is a write into a shared buffer that the r
 * receivers read.  A kernel acting for node k dereferences node k's buffers
 * and the shared coded buffer only.
 *
 * Conventions
 *   - Every function returns CCDC_OK (0) or a negative ccdc_status; nothing
 *     throws, aborts or traps.  Arguments are validated before any launch.
 *   - The library owns only the plan (host tables and, after the first device
 *     call or ccdc_plan_upload, their device copies on the device that was
 *     current then).  The caller owns every data buffer and the stream.
 *   - "device pointer array": a HOST array of K pointers to DEVICE memory,
 *     entry k belonging to node k.  Data pointers must be 16-byte aligned.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     All step functions are asynchronous on it; a step that follows another
 *     on the same stream sees its results.
 *   - A plan may be used by one host thread at a time and on one device: the
 *     device that was current when its tables were uploaded (another device
 *     gives CCDC_ESTATE).  Different plans are independent.
 *   - Elements are 32 bits wide: int32 with wrapping addition or IEEE binary32.
 *     XOR coding acts on the raw bit patterns in both cases.
 *
 * Layouts (element = 32-bit word; len = (Q/K)*B; s = ceil(len / r))
 *   partition of node k   [local batch][file in batch][q = 0..Q-1][B]
 *                         local batches = the batches whose label contains k,
 *                         in ascending batch id; files ascending.
 *   packets of node k     [local batch][outside node t, ascending][len]
 *                         (stepwise API only)
 *   coded buffer          [round][sender rank inside the round's subset][s_pad]
 *                         s_pad = s rounded up to a multiple of 4 words; only
 *                         the first s words of a row are multicast bits.
 *   decoded of node k     [rounds that contain k, ascending][len]
 *                         (stepwise API only)
 *   out                   [job][q = 0..Q-1][B]; function q belongs to node
 *                         q / (Q/K).
 */
#ifndef CCDC_H
#define CCDC_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ccdc_plan_s ccdc_plan_t;     /* opaque; created and destroyed by the library */

typedef enum { CCDC_I32 = 0, CCDC_F32 = 1 } ccdc_dtype_t;

typedef enum {
    CCDC_OK = 0,
    CCDC_EINVAL = -1,   /* parameters outside the paper's setting, NULL or misaligned pointer */
    CCDC_ENOMEM = -2,   /* host or device allocation of plan tables failed */
    CCDC_ECUDA = -3,    /* a CUDA call or launch failed; see ccdc_last_cuda_error */
    CCDC_ESIZE = -4,    /* a size exceeds what the entry point supports */
    CCDC_ESTATE = -5    /* call not valid for this plan (e.g. ccdc_map on a plan without a Map) */
} ccdc_status;

#define CCDC_MAX_K 32   /* nodes; the subset tables grow as C(K, r+1) */

/* ------------------------------------------------------------------ plan
 * Section IV-A (file placement), Section III (function assignment S_k) and the
 * multicast schedule of Section IV-B.
 *
 * ccdc_plan: ONE job over all K nodes.  The N files are cut into C(K,r)
 * batches of b = N / C(K,r) consecutive files; batch p is labelled by the p-th
 * size-r subset of {0..K-1} in lexicographic order and stored at those r
 * nodes.  There is one multicast round per size-(r+1) subset S (lexicographic):
 * member t of S receives the batch labelled S\{t}.  Node k reduces functions
 * k*Q/K .. (k+1)*Q/K-1.
 *   requires 2 <= K <= CCDC_MAX_K, 1 <= r <= K-1, K <= N, C(K,r) | N, K | Q,
 *   B >= 1; otherwise CCDC_EINVAL and *out = NULL.  CCDC_ESIZE when the schedule
 *   is too large to tabulate (more than 2^24 rounds, or decode tables beyond 2 GB).
 *
 * ccdc_plan_jobs: the scheme as Section IV states it for J = C(K,r+1) jobs
 * (gamma = 1).  Job j lives on the j-th size-(r+1) subset K_j; its N files are
 * cut into r+1 batches labelled by the size-r subsets of K_j (lexicographic).
 * Rounds, for each subset S = K_j in order: stage 1, then one stage-2 round
 * per outside node i ascending, in which member t receives the batch labelled
 * S\{t} of the job living on {i} U S\{t}.  Global file id = j*N + n; global
 * function id = j*Q + q.   requires additionally (r+1) | N.
 *
 * Host only: no CUDA call is made.  Destroy with ccdc_plan_destroy. */
int  ccdc_plan(int K, int r, long long N, int Q, long long B, ccdc_dtype_t dtype, ccdc_plan_t **out);
int  ccdc_plan_jobs(int K, int r, long long N, int Q, long long B, ccdc_dtype_t dtype, ccdc_plan_t **out);
/* ccdc_plan_jobs_gamma: J = gamma * C(K,r+1) jobs (Section IV: "repeats the same
 * operations gamma times"), all shuffled by the same two launches.  Job j lives
 * on subset j mod C(K,r+1); jobs g*C(K,r+1) .. (g+1)*C(K,r+1)-1 form group g, an
 * independent instance of ccdc_plan_jobs whose batches, rounds, files (global id
 * j*N + n), functions and outputs follow those of group g-1 in every layout.
 * gamma >= 1 (CCDC_EINVAL otherwise); gamma = 1 is ccdc_plan_jobs. */
int  ccdc_plan_jobs_gamma(int K, int r, long long N, int Q, long long B, ccdc_dtype_t dtype, int gamma,
                          ccdc_plan_t **out);
/* ccdc_plan_compression: the compression-only scheme of the paper's appendix
 * ("Communication Load of the compression scheme"), kept as a measured
 * comparator.  One job, mu = r/K: the files are cut into m = ceil(K/r) batches,
 * the first m-1 of mu*N files and the last of the rest; node k stores batch
 * k mod m (so its partition is [file in batch][q][B] with ccdc_plan_batch_files
 * files); for every batch t it lacks, node k is sent ONE pre-combined packet of
 * its Q/K functions by the first node after k, cyclically, that stores batch t
 * (the paper leaves the sender open).  No coding: only ccdc_compression_shuffle
 * and ccdc_reduce accept such a plan, the coded steps return CCDC_ESTATE.
 * ccdc_plan_coded_bits is then the unicast bit count K*(m-1)*32*len, i.e. the
 * load ceil(1/mu)-1 of Eq. (2).   requires additionally K | r*N.
 * Queries: ccdc_plan_num_batches = m, ccdc_plan_num_groups = 0, holders of a
 * batch are reported in r slots padded with -1. */
int  ccdc_plan_compression(int K, int r, long long N, int Q, long long B, ccdc_dtype_t dtype, ccdc_plan_t **out);
/* ccdc_plan_sharded: the plan of ccdc_plan (jobs = 0) or ccdc_plan_jobs (jobs != 0)
 * restricted to the logical nodes of one GPU out of `world` (the broadcast
 * network of Section III becomes an all-gather between GPUs).  Requires
 * world | K; node k lives on rank k / (K/world).  On such a plan
 *   - pointer arrays still have K entries; only this rank's nodes are used;
 *   - ccdc_encode_fused writes only the coded rows this rank's nodes send, packed
 *     into a send buffer of ccdc_coded_send_bytes (the same on every rank);
 *   - the caller gathers the send buffers of all ranks, rank-major, into a buffer
 *     of ccdc_coded_bytes (e.g. ncclAllGather / all_gather_into_tensor): coded row
 *     (round g, sender rank a) is then row ccdc_plan_coded_row_position(plan, g, a);
 *   - ccdc_decode_reduce reads that gathered buffer and writes only the outputs of
 *     this rank's nodes (out keeps its full [job][q][B] layout);
 *   - ccdc_map maps only this rank's files; ccdc_shuffle and the stepwise calls
 *     return CCDC_ESTATE.
 * The bytes that cross between GPUs are the multicast bits of the scheme:
 * ccdc_plan_coded_bits / 8 in total, each rank contributing 1/world. */
int  ccdc_plan_sharded(int K, int r, long long N, int Q, long long B, ccdc_dtype_t dtype, int jobs, int rank,
                       int world, ccdc_plan_t **out);
long long ccdc_plan_coded_row_position(const ccdc_plan_t *plan, long long g, int a);
int  ccdc_plan_node_is_local(const ccdc_plan_t *plan, int k);
size_t ccdc_coded_send_bytes(const ccdc_plan_t *plan);
void ccdc_plan_destroy(ccdc_plan_t *plan);

/* Copies the schedule tables to the current device (cudaMalloc + cudaMemcpy,
 * synchronous).  Optional: the first step call on a plan does it implicitly.
 * After it no step function allocates.  CCDC_ENOMEM / CCDC_ECUDA on failure.
 * The launch shapes of a plan are sized for 148 SMs (B200) when it is created;
 * the upload sizes them again for the current device's SM count, which can
 * change ccdc_workspace_bytes on another GPU model: query it after the upload
 * there. */
int  ccdc_plan_upload(ccdc_plan_t *plan);

/* Kernel family of the fused encode and decode: 0 = loads through registers
 * (any plan; the planner's choice for every plan, it measured faster on every
 * workload), 1 = bulk-copy pipelines: the lanes of one warp per block stream
 * whole operand rows into a ring of shared-memory stages with asynchronous bulk
 * copies and the other threads fold them (needs 4 | (Q/K)*B, 2 | s and a
 * device of compute capability >= 9; CCDC_ESIZE otherwise).
 * ccdc_plan_tune_family selects a family, before the tables are uploaded
 * (CCDC_ESTATE after), and re-sizes the split of the decode for it.  Both
 * families add in the same order and give the same bits.  The waits of family 1
 * are bounded; ccdc_shuffle_status (call it after synchronising the stream;
 * copies one word back) returns CCDC_ESTATE if one ever ran out on this plan,
 * in which case that call's outputs are not valid. */
int  ccdc_plan_kernel_family(const ccdc_plan_t *plan);
int  ccdc_plan_tune_family(ccdc_plan_t *plan, int family);
int  ccdc_shuffle_status(const ccdc_plan_t *plan);

/* Launch shape of the fused decode (ccdc_decode_reduce), chosen by the planner:
 * threads per block, and the number of blocks (chunks) the loop over a job's
 * batches is split into (1 = no workspace needed).
 * ccdc_plan_decode_cluster: 1 if the blocks that share an output tile (one per
 * chunk) form a thread-block cluster and add their partial sums through
 * distributed shared memory, in chunk order: then ccdc_workspace_bytes is 0 and
 * ccdc_decode_reduce is a single launch.  Chosen for 2..8 chunks on plans with
 * several files per batch (r <= 4, even segment length); other split plans use
 * the workspace and a second small launch.
 * ccdc_plan_tune_decode overrides the planner's choice, e.g. from a timing
 * sweep; it changes ccdc_workspace_bytes.  Allowed: chunks in 1..batches per
 * job; threads 128 for plans with several files per batch, r <= 4 and an even
 * segment length, else 512 or 1024 (CCDC_EINVAL otherwise); only before the
 * tables are uploaded (CCDC_ESTATE after).  Results do not depend on the shape
 * for int32; for fp32 the grouping of the per-batch terms follows the chunks
 * (Eq. (1) is a sum). */
int  ccdc_plan_decode_threads(const ccdc_plan_t *plan);
int  ccdc_plan_decode_chunks(const ccdc_plan_t *plan);
int  ccdc_plan_decode_cluster(const ccdc_plan_t *plan);
int  ccdc_plan_tune_decode(ccdc_plan_t *plan, int threads, int chunks);

/* ---------------------------------------------------------------- queries
 * All host side, valid for the plan's lifetime.  Index arguments out of range
 * give CCDC_EINVAL (or 0 for the size queries). */
long long ccdc_plan_num_jobs(const ccdc_plan_t *plan);        /* J */
long long ccdc_plan_num_batches(const ccdc_plan_t *plan);     /* over all jobs */
long long ccdc_plan_num_groups(const ccdc_plan_t *plan);      /* multicast rounds: C(K,r+1) per job batch set */
long long ccdc_plan_files_per_batch(const ccdc_plan_t *plan); /* b */
long long ccdc_plan_batch_files(const ccdc_plan_t *plan, long long p); /* files in batch p (differs from b only
                                                                           for the last batch of a compression plan) */
long long ccdc_plan_packet_elems(const ccdc_plan_t *plan);    /* len = (Q/K)*B */
long long ccdc_plan_segment_elems(const ccdc_plan_t *plan);   /* s = ceil(len/r) */
long long ccdc_plan_coded_row_elems(const ccdc_plan_t *plan); /* s_pad */
/* exact number of bits multicast: rounds * (r+1) * 32 * s  (Definition 1 counts a broadcast once) */
long long ccdc_plan_coded_bits(const ccdc_plan_t *plan);
/* nodes_out[r]: ascending ids of the nodes storing global file n */
int  ccdc_plan_batch_of_file(const ccdc_plan_t *plan, long long n, int *nodes_out);
/* nodes_out[r] = label of batch p; *first_file = its first global file id; *job = its job */
int  ccdc_plan_batch(const ccdc_plan_t *plan, long long p, int *nodes_out, long long *first_file, long long *job);
/* members_out[r+1]: ascending node ids of round g */
int  ccdc_plan_group(const ccdc_plan_t *plan, long long g, int *members_out);
/* batches_out[r+1]: batch id whose packet member a of round g receives */
int  ccdc_plan_group_batches(const ccdc_plan_t *plan, long long g, long long *batches_out);
/* number of batches stored at node k, and their ids (ascending) into ids_out (may be NULL) */
long long ccdc_plan_node_batches(const ccdc_plan_t *plan, int k, long long *ids_out);

size_t ccdc_partition_bytes(const ccdc_plan_t *plan, int k);  /* node k's Map results */
size_t ccdc_packets_bytes(const ccdc_plan_t *plan, int k);    /* stepwise API */
size_t ccdc_decoded_bytes(const ccdc_plan_t *plan, int k);    /* stepwise API */
size_t ccdc_coded_bytes(const ccdc_plan_t *plan);             /* shared multicast buffer */
size_t ccdc_out_bytes(const ccdc_plan_t *plan);               /* J*Q*B*4 */
size_t ccdc_workspace_bytes(const ccdc_plan_t *plan);         /* ccdc_shuffle scratch; may be 0 */

/* ------------------------------------------------------------------ steps
 * part, packets, decoded: device pointer arrays (see above). */

/* Map phase (Section III, "Map phase") of the linear-regression workload: for
 * every file n stored at node k, the Q intermediate values v_{q,n} are the Q
 * contiguous slices of the partial gradient
 *     g_n = X_n^T (X_n w - y_n),   X_n [rows][d] bf16 row-major, d = Q*B,
 *     y_n [rows] fp32, w [d] bf16,
 * computed with bf16 tensor-core products accumulated in fp32 (the fp32
 * residual enters the second product as the sum of three bf16 terms, so no
 * precision is lost to the operand format) and written as fp32 into part[k] in
 * the partition layout.  Every node maps its own copy of a file; replicas are
 * bit-identical because the same deterministic kernels, with one fixed
 * summation order, run for each.
 *   files_x[k]: node k's files, [local batch][file in batch][rows][d] bf16
 *   files_y[k]: [local batch][file in batch][rows] fp32
 *   w: device pointer, [d] bf16;  workspace: ccdc_map_workspace_bytes(plan, rows)
 *   (residuals plus a few control words; the call resets what it needs).
 * F32 plans only (CCDC_ESTATE otherwise).  CCDC_ESIZE unless rows is a multiple
 * of 16 in 16..4096 and d a multiple of 512 up to 65536.  Asynchronous on
 * `stream`: one memset and one or two kernel launches.
 *
 * Which kernel runs (ccdc_map_last_kernel tells):
 *  - d = 2048, 4096, 8192 or 16384: a thread-block cluster of d/2048 blocks owns a
 *    file, each block 2048 columns.  X is staged by TMA into a ring of
 *    shared-memory stages (8 rows x 2048 columns each) and read from HBM exactly
 *    once: both products of a row block run from the same stage, the blocks of a
 *    cluster exchanging their partial dot products through distributed shared
 *    memory.  Files are cut into units of rows/4 rows (when rows is a multiple of
 *    32) that are shared out evenly over the clusters; a file's gradient is always
 *    ((unit0 + unit1) + unit2) + unit3, whichever clusters computed the units, so
 *    replicas stay bit-identical; files cut between two clusters are summed by a
 *    small second launch from the workspace.  All waits (mbarrier polls) are
 *    bounded.
 *  - other shapes, or a device or driver without tensor maps or room for the
 *    cluster: loads through registers; work items are handed out in order by an
 *    atomic ticket (per file its first-product blocks, then the second-product
 *    blocks of an earlier file) so that the second product finds the file in L2;
 *    a second-product block polls a per-file counter until the file's residuals
 *    are complete.  The blocks it waits for hold smaller tickets, are therefore
 *    already running and wait on nothing, so the poll always ends; it is bounded
 *    anyway.
 * ccdc_map_status reports if a bound was ever hit in either kernel.
 *
 * ccdc_map_status: call after the stream has been synchronised; copies one word
 * back (synchronous) and returns CCDC_OK, or CCDC_ESTATE if a wait ran out (the
 * Map results of that call are then not valid). */
size_t ccdc_map_workspace_bytes(const ccdc_plan_t *plan, long long rows);
int ccdc_map(ccdc_plan_t *plan, const void *const *files_x, const void *const *files_y, const void *w,
             long long rows, void *const *part, void *workspace, void *stream);
int ccdc_map_status(const ccdc_plan_t *plan, long long rows, const void *workspace);
/* Name of the kernel the most recent ccdc_map of this process launched ("k_map_cluster": X staged by
 * TMA through a thread-block cluster, read once; "k_map": loads through registers, for shapes or
 * devices the first cannot serve; "" before the first call).  Static string, not thread safe. */
const char *ccdc_map_last_kernel(void);

/* Pre-combining (Section IV-B): packets[k][local batch][t] = concatenation over
 * q in S_t of  sum_{n in batch} v_{q,n}, files added in ascending order
 * starting from the first file's value. */
int ccdc_combine(ccdc_plan_t *plan, const void *const *part, void *const *packets, void *stream);

/* Encoding (Section IV-B, message X_k): coded[round][a] = XOR over the other
 * members t of the round of segment (label = sender) of the sender's packet
 * for t; segments are s words, the last one zero extended. */
int ccdc_encode(ccdc_plan_t *plan, const void *const *packets, void *coded, void *stream);

/* Decoding (Section IV-B): for every node k, round containing k and sender
 * k' != k: coded packet XOR the r-1 segments labelled k' of k's own packets
 * for the other members = segment labelled k' of the packet meant for k. */
int ccdc_decode(ccdc_plan_t *plan, const void *const *packets, const void *coded,
                void *const *decoded, void *stream);

/* Reduce (Eq. (1), final reduction of Section IV): out[j][q] = sum over the
 * batches of job j, ascending, of the local pre-combined value (batch stored at
 * the node of q) or the decoded one. */
int ccdc_reduce(ccdc_plan_t *plan, const void *const *part, const void *const *decoded,
                void *out, void *stream);

/* The four steps fused into two launches (plus a small deterministic final
 * pass when the batch loop is split): pre-combining is recomputed inside the
 * encode and inside the decode, decoded packets are never stored, every value
 * a node needs is read from its partition once.
 *
 * ccdc_encode_fused: launch 1.  coded[round][a] straight from the sender's
 *   partition (pre-combining of Section IV-B + message X_k).  Bit-identical to
 *   ccdc_combine followed by ccdc_encode.
 * ccdc_decode_reduce: launch 2.  For node k, each of its output words: over
 *   the batches of the job in ascending order, the local pre-combined word, or
 *   the coded word XOR the r-1 cancellable pre-combined words (decoding of
 *   Section IV-B), accumulated as Eq. (1) demands.  When the loop over the
 *   batches is split over several blocks, the partial sums are added in chunk
 *   order: inside a thread-block cluster (ccdc_plan_decode_cluster), or from
 *   the workspace by a second small launch.  workspace:
 *   ccdc_workspace_bytes (may be NULL if that is 0); it is fully overwritten
 *   before it is read.  int32 outputs are
 *   bit-identical to the stepwise path; fp32 outputs are too when the
 *   workspace size is 0, and otherwise differ from it only by the grouping of
 *   the per-batch terms.
 * ccdc_shuffle: both, in order, on `stream`.
 *   coded: ccdc_coded_bytes; out: ccdc_out_bytes.
 * These calls (and ccdc_shuffle) enqueue kernels only, so they can be captured in
 * a CUDA graph once the plan's tables are on the device (after ccdc_plan_upload
 * or a first call). */
int ccdc_encode_fused(ccdc_plan_t *plan, const void *const *part, void *coded, void *stream);
int ccdc_decode_reduce(ccdc_plan_t *plan, const void *const *part, const void *coded, void *out,
                       void *workspace, void *stream);

/* Encode fused with the exchange between GPUs (node-sharded plans only, else
 * CCDC_ESTATE): the multicast of Section IV-B done by the producing kernel.
 * peer_coded: HOST array of `world` device pointers, entry d = rank d's full
 * coded buffer (ccdc_coded_bytes) as addressable from this GPU (its own buffer
 * for d = this rank, peer mappings for the others).  Every coded row this rank's
 * nodes send is stored straight into its gathered position in all `world`
 * buffers, so no separate all-gather is needed; the ranks must still synchronise
 * (on the host, or with stream events) before any of them launches
 * ccdc_decode_reduce, because a kernel of one rank never waits for another
 * rank.  Needs one file per batch or r <= 4 operands (CCDC_ESIZE otherwise). */
int ccdc_encode_fused_peers(ccdc_plan_t *plan, const void *const *part, void *const *peer_coded, void *stream);
int ccdc_shuffle(ccdc_plan_t *plan, const void *const *part, void *coded, void *out,
                 void *workspace, void *stream);

/* The appendix's compression-only shuffle (comparator; plans from
 * ccdc_plan_compression only, else CCDC_ESTATE).  recv: device pointer array,
 * recv[k] = ccdc_decoded_bytes(plan, k) = the m-1 packets node k receives,
 * batches ascending.  Launch 1: every packet = sum over the sender's batch of
 * the receiver's Q/K values (files ascending, starting from the first file's
 * value), written to the receiver's buffer.  Launch 2: Eq. (1): batches
 * ascending, the node's own batch from its partition, the others from recv. */
int ccdc_compression_shuffle(ccdc_plan_t *plan, const void *const *part, void *const *recv, void *out,
                             void *stream);

/* ccdc_shuffle on Map results that live in HOST memory (Section III: the
 * Shuffle phase starts from each node's local Map results and ends with the
 * Reduce outputs at the nodes).  host_part: host array of K HOST pointers,
 * node k's partition (ccdc_partition_bytes(k); pinned memory makes the copies
 * asynchronous); host_out: HOST buffer of ccdc_out_bytes.  dev_part, dev_coded,
 * dev_out, dev_workspace: device staging buffers of the usual sizes, owned by
 * the caller.  Enqueues on `stream`: K host-to-device copies, the two
 * launches, one device-to-host copy of the outputs; returns without waiting. */
int ccdc_shuffle_host(ccdc_plan_t *plan, const void *const *host_part, void *host_out,
                      void *const *dev_part, void *dev_coded, void *dev_out, void *dev_workspace,
                      void *stream);

/* The same from Map results that sit in host memory ONCE per file: host_values is
 * [J*N files][Q][B] in global file order (pinned memory makes the copies
 * asynchronous).  Every file is copied to the device once, into the partition of
 * the first node that stores it (Section IV-A placement), and from there, device
 * to device, into the partitions of the other r-1 nodes that store it -- the
 * replicas of a file are bit-identical by the scheme's own premise -- so the
 * host-to-device traffic is N*Q*B words instead of r times that.  Then
 * ccdc_shuffle and one device-to-host copy of the outputs.  Plans from ccdc_plan,
 * ccdc_plan_jobs and ccdc_plan_jobs_gamma (CCDC_ESTATE otherwise).  Enqueues on
 * `stream` (r copy calls per batch of files) and returns without waiting. */
int ccdc_shuffle_host_files(ccdc_plan_t *plan, const void *host_values, void *host_out, void *const *dev_part,
                            void *dev_coded, void *dev_out, void *dev_workspace, void *stream);

/* A whole linear-regression job from HOST memory (Section III: Map phase, Shuffle
 * phase, Reduce outputs): copies node k's files host_x[k] ([files][rows][d] bf16),
 * host_y[k] ([files][rows] fp32) and host_w ([d] bf16) into the device staging
 * buffers dev_x[k], dev_y[k], dev_w, then ccdc_map into dev_part, ccdc_shuffle,
 * and one device-to-host copy of the outputs into host_out (ccdc_out_bytes).
 * All device buffers are the caller's, of the sizes the separate calls take
 * (map_workspace: ccdc_map_workspace_bytes; dev_workspace: ccdc_workspace_bytes).
 * Pinned host memory makes the copies asynchronous.  Enqueues on `stream` and
 * returns without waiting; errors as ccdc_map and ccdc_shuffle. */
int ccdc_job_host(ccdc_plan_t *plan, const void *const *host_x, const void *const *host_y, const void *host_w,
                  long long rows, void *host_out, void *const *dev_x, void *const *dev_y, void *dev_w,
                  void *const *dev_part, void *dev_coded, void *dev_out, void *map_workspace, void *dev_workspace,
                  void *stream);

/* --------------------------------------------------------- several GPUs
 * One process per GPU.  The shuffle shards two ways; neither makes a kernel of
 * one GPU wait for another GPU.
 *
 * (1) Value-dimension shards, no exchange.  Every step of Section IV-B (sums,
 * XORs, cancellations) acts on words at equal positions of equal-size
 * segments, so GPU `rank` of `world` can own the sub-range [rank*w, (rank+1)*w),
 * w = s/world, of EVERY segment of every packet and run the complete scheme on
 * it: an exact instance of the scheme with values of B_local = r*w/(Q/K)
 * elements.  Requires r | (Q/K)*B, world | s and (Q/K) | r*w (CCDC_EINVAL
 * otherwise).  Each rank makes an ordinary plan ccdc_plan(K, r, N, Q, B_local)
 * (or ccdc_plan_jobs) and shuffles alone; the multicast bits of the ranks add
 * up to those of the unsharded job.
 *   ccdc_value_shard           B_local for this rank (host only).
 *   ccdc_value_shard_position  position in the full packet ((Q/K)*B words) of
 *                              word local_pos of the rank's packet (r*w words);
 *                              -1 if out of range (host only).
 *   ccdc_value_shard_copy      device copy between the full layout
 *                              [rows][Q][B] and the rank's [rows][Q][B_local]
 *                              (rows = files for Map results, jobs for
 *                              outputs): to_local != 0 gathers the rank's words
 *                              out of `src` (full) into `dst` (local); to_local
 *                              = 0 scatters `src` (local) to the rank's
 *                              positions of `dst` (full), leaving the rest of
 *                              dst untouched.  One launch on `stream`.  A Map
 *                              that runs per rank would write its slice
 *                              directly; the copy serves tests and callers
 *                              that hold full-length values. */
int ccdc_value_shard(int K, int r, int Q, long long B, int rank, int world, long long *B_local);
long long ccdc_value_shard_position(int K, int r, int Q, long long B, int rank, int world, long long local_pos);
int ccdc_value_shard_copy(int K, int r, int Q, long long B, int rank, int world, int to_local, const void *src,
                          void *dst, long long rows, void *stream);

/* (2) Node shards with peer stores (ccdc_plan_sharded + ccdc_encode_fused_peers,
 * above): the multicast of Section IV-B as plain stores into every rank's coded
 * buffer.  For that each rank's buffer must be addressable from the other
 * processes: ccdc_peer_buffer_create allocates `bytes` of device memory on the
 * current device and fills handle_out (CCDC_PEER_HANDLE_BYTES bytes, to be sent
 * to the other ranks by any host channel); ccdc_peer_buffer_open maps another
 * process's buffer into this one (peer access is enabled as needed) and
 * ccdc_peer_buffer_close unmaps it; ccdc_peer_buffer_destroy frees one's own
 * buffer after the others closed it.  ccdc_peer_buffer_copy is an asynchronous
 * copy between any two of device, peer and host memory (direction inferred).
 * These calls allocate and synchronise: set-up and tear-down, not the data
 * path.  The data path stays plain peer stores by the encode kernel; the ranks
 * synchronise on the host (or with a collective on the stream) between the
 * encode and the decode launch. */
#define CCDC_PEER_HANDLE_BYTES 64
int ccdc_peer_buffer_create(size_t bytes, void **dev_ptr, void *handle_out);
int ccdc_peer_buffer_open(const void *handle, void **dev_ptr);
int ccdc_peer_buffer_close(void *dev_ptr);
int ccdc_peer_buffer_destroy(void *dev_ptr);
int ccdc_peer_buffer_copy(void *dst, const void *src, size_t bytes, void *stream);

/* Allocation-free variant of ccdc_decode_reduce (the paper has no counterpart:
 * this is a property of the library, not a step of the scheme).
 *
 * For callers that cannot allocate device memory where they shuffle -- code in
 * a region where cudaMalloc is forbidden or would stall the device, or a
 * program whose memory was handed out in full at start-up.  The scratch of the
 * split batch loop is a fixed array of ccdc_static_scratch_bytes() (16 MiB) of
 * device memory inside the library image; every GPU that loads the library
 * holds it until the process exits.  The caller still passes inputs and
 * outputs; results are identical to ccdc_decode_reduce.
 *   - makes no cudaMalloc / cudaFree / allocating library call.  The plan's
 *     tables must already be on the current device (ccdc_plan_upload, done
 *     earlier by code that may allocate); otherwise CCDC_ESTATE.
 *   - CCDC_ESIZE if ccdc_workspace_bytes(plan) exceeds the array.
 *   - the first call on a device looks up the array's device address (once per
 *     device, with that device current); make that first call before starting
 *     any stream capture.
 *   - all calls on a device share the array and it keeps the previous call's
 *     contents; the kernels overwrite every word they later read, so nothing
 *     needs clearing, but two calls whose kernels overlap on the GPU (different
 *     streams, different plans or threads) race on it: serialise them. */
size_t ccdc_static_scratch_bytes(void);
int ccdc_decode_reduce_static(ccdc_plan_t *plan, const void *const *part, const void *coded, void *out,
                              void *stream);

/* ------------------------------------------------------------- diagnostics */
const char *ccdc_strerror(int status);
int ccdc_last_cuda_error(void);          /* cudaError_t of the last CCDC_ECUDA on this thread */
int ccdc_num_kernel_launches(void);      /* kernels launched by this library so far (process wide) */
/* Which kernel form the calling thread's most recent gather launch (ccdc_combine, ccdc_encode,
 * ccdc_decode, ccdc_encode_fused, the first launch of ccdc_compression_shuffle) and most recent
 * ccdc_decode_reduce used, e.g. "k_gather_static<vec=4,operands=2,files=1,vectors=2,threads=512>";
 * "" before the first.  Static per-thread strings. */
const char *ccdc_last_gather_kernel(void);
const char *ccdc_last_decode_kernel(void);

#ifdef __cplusplus
}
#endif
#endif /* CCDC_H */
