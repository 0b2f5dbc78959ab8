// CUDA kernels (sm_100a) and launch code of the compressed CDC shuffle.
//
// All steps are streaming: at most one add or XOR per 32-bit word moved, so
// the kernels are organised around wide coalesced loads with many independent
// loads in flight per thread, and tables of element offsets prepared by the
// host planner.  A thread block that works for node k reads node k's buffers
// and the shared coded buffer only.
//
//   k_gather_static   a destination row = XOR over a compile-time number of
//                     operands of the batch sums of a segment (the fused encode,
//                     the stepwise combine and encode, the compression-only
//                     unicast with its per-row file counts); loads in registers
//   k_gather          the same for any operand count and with a coded input row
//                     (r > 4, the stepwise decode); cp.async pipeline through
//                     shared memory
//   k_decode_reduce   decode + cancel + reduce, decoded packets never stored
//   k_sum_chunks      ordered sum of the partial outputs when the batch loop
//                     of k_decode_reduce is split over blocks through the workspace
//   k_reduce          Eq. (1) from materialised packets (stepwise API)
// No kernel here spins on memory another block or thread writes: the
// encode -> decode dependency is the boundary between two launches on one
// stream (each kernel starts behind griddepcontrol.wait, a dependency the
// hardware resolves), and the one place blocks meet inside a kernel, the
// clustered decode, uses the hardware barrier of a thread-block cluster.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <cstdio>
#include <algorithm>
#include <cstring>
#include <type_traits>
#include <utility>

#include "ccdc_internal.h"
#include "ccdc_stream.h"

namespace {

// launch shapes: D* = fused decode+reduce and the stepwise reduce, G* = gather
constexpr int DTHREADS = CCDC_DECODE_THREADS;
constexpr int DUNROLL = CCDC_DECODE_VECTORS;
constexpr int GTHREADS = CCDC_GATHER_THREADS;
constexpr int GUNROLL = CCDC_GATHER_VECTORS;
constexpr int STAGES = CCDC_GATHER_STAGES;

thread_local int g_last_cuda_error = 0;
thread_local char g_last_gather[96] = "";     // the instantiations this thread launched last
thread_local char g_last_decode[96] = "";
std::atomic<int> g_launches{0};

int cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int)e;
    return CCDC_ECUDA;
}

// ------------------------------------------- programmatic dependent launch
// Every kernel here is launched so that the GPU may schedule its blocks while
// the previous kernel of the stream is still draining: it first lets its own
// dependent go (pdl_trigger), reads what no kernel writes (the plan's tables),
// and calls pdl_wait -- which returns once the previous kernel has finished and
// its writes are visible -- before it touches any data buffer.  Nothing is read
// or written before the wait except plan tables, so the order of the stream is
// kept exactly; what is saved is the launch latency between short kernels.
// (A hardware dependency of the launch, not a spin: there is nothing to time out.)
#ifndef CCDC_USE_PDL
#define CCDC_USE_PDL 1
#endif
__device__ __forceinline__ void pdl_trigger() {
#if CCDC_USE_PDL
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
#endif
}
__device__ __forceinline__ void pdl_wait() {
#if CCDC_USE_PDL
    asm volatile("griddepcontrol.wait;" ::: "memory");
#endif
}

// cluster > 1: consecutive groups of `cluster` blocks form a thread-block cluster
template <typename... KArgs, typename... Args>
cudaError_t launch_clustered(void (*kernel)(KArgs...), int cluster, long long grid, int block, size_t smem, cudaStream_t st,
                             Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n = 0;
    if (CCDC_USE_PDL) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    if (cluster > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = (unsigned)cluster;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

template <typename... KArgs, typename... Args>
cudaError_t launch_kernel(void (*kernel)(KArgs...), long long grid, int block, size_t smem, cudaStream_t st, Args &&...args) {
    return launch_clustered(kernel, 1, grid, block, smem, st, std::forward<Args>(args)...);
}

// ---- thread-block clusters: barrier over the blocks of a cluster, loads from a peer block's shared memory
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ unsigned peer_shared_address(const void *local, unsigned rank) {
    unsigned remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"((unsigned)__cvta_generic_to_shared(local)), "r"(rank));
    return remote;
}

// ---------------------------------------------------------------- vectors
template <int VEC> struct WordVec;
template <> struct WordVec<1> { using type = unsigned int; };
template <> struct WordVec<2> { using type = uint2; };
template <> struct WordVec<4> { using type = uint4; };

template <int VEC> struct Words { uint32_t w[VEC]; };

template <int VEC>
__device__ __forceinline__ Words<VEC> load_words(const uint32_t *p) {
    using V = typename WordVec<VEC>::type;
    V v = __ldg(reinterpret_cast<const V *>(p));
    Words<VEC> out;
    memcpy(out.w, &v, sizeof(V));
    return out;
}

template <int VEC>
__device__ __forceinline__ void store_words(uint32_t *p, const Words<VEC> &x) {
    using V = typename WordVec<VEC>::type;
    V v;
    memcpy(&v, x.w, sizeof(V));
    *reinterpret_cast<V *>(p) = v;
}

// VEC words from the shared memory of block `rank` of this block's cluster, at the slot `local` names here
template <int VEC>
__device__ __forceinline__ Words<VEC> load_words_peer(const uint32_t *local, unsigned rank) {
    const unsigned a = peer_shared_address(local, rank);
    Words<VEC> out;
    if constexpr (VEC == 4)
        asm volatile("ld.shared::cluster.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(out.w[0]), "=r"(out.w[1]), "=r"(out.w[2]), "=r"(out.w[3]) : "r"(a));
    else if constexpr (VEC == 2)
        asm volatile("ld.shared::cluster.v2.u32 {%0,%1}, [%2];" : "=r"(out.w[0]), "=r"(out.w[1]) : "r"(a));
    else
        asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(out.w[0]) : "r"(a));
    return out;
}

template <int VEC>
__device__ __forceinline__ Words<VEC> zero_words() {
    Words<VEC> z;
#pragma unroll
    for (int i = 0; i < VEC; ++i) z.w[i] = 0u;
    return z;
}

// the aggregation of Eq. (1): int32 wrapping add, or IEEE binary32 add
template <bool F32>
__device__ __forceinline__ uint32_t add_word(uint32_t a, uint32_t b) {
    if (F32) return __float_as_uint(__fadd_rn(__uint_as_float(a), __uint_as_float(b)));
    return a + b;
}

template <int VEC, bool F32>
__device__ __forceinline__ void add_into(Words<VEC> &a, const Words<VEC> &b) {
#pragma unroll
    for (int i = 0; i < VEC; ++i) a.w[i] = add_word<F32>(a.w[i], b.w[i]);
}

template <int VEC>
__device__ __forceinline__ void xor_into(Words<VEC> &a, const Words<VEC> &b) {
#pragma unroll
    for (int i = 0; i < VEC; ++i) a.w[i] ^= b.w[i];
}

// sum over the b files of a batch, ascending, starting from the first file's
// value (pre-combined value of Section IV-B); zero where the segment does not exist
template <int VEC, bool F32>
__device__ __forceinline__ Words<VEC> batch_sum(const uint32_t *src, long long off, long long j,
                                                long long vl, int b, long long file_stride) {
    if (j >= vl) return zero_words<VEC>();
    const uint32_t *p = src + off + j;
    Words<VEC> acc = load_words<VEC>(p);
    for (int f = 1; f < b; f += 4) {        // up to four files' loads in flight, added in file order
        Words<VEC> w[4];
#pragma unroll
        for (int x = 0; x < 4; ++x)
            if (f + x < b) w[x] = load_words<VEC>(p + (long long)(f + x) * file_stride);
#pragma unroll
        for (int x = 0; x < 4; ++x)
            if (f + x < b) add_into<VEC, F32>(acc, w[x]);
    }
    return acc;
}

// ------------------------------------------------- asynchronous load pipeline
// Every streaming kernel keeps STAGES chunks of global loads in flight per
// thread without holding them in registers: a thread copies its own VEC words
// of a chunk global -> shared with cp.async (no register staging, the thread
// runs on), commits one group per chunk, and STAGES-1 chunks later waits for
// that group and reads its own words back.  A thread only ever reads slots it
// filled itself, so the data path needs no block-wide barrier, and nothing
// here can wait on another thread: there is no flag or mbarrier to hang on.

template <int VEC>
__device__ __forceinline__ void async_copy(uint32_t *smem, const uint32_t *gmem) {
    const unsigned addr = (unsigned)__cvta_generic_to_shared(smem);
    if (VEC == 4) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(addr), "l"(gmem) : "memory");
    else if (VEC == 2) asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(addr), "l"(gmem) : "memory");
    else asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(addr), "l"(gmem) : "memory");
}
__device__ __forceinline__ void async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory"); }

// this thread's slot for vector u of a stage
template <int VEC>
__device__ __forceinline__ uint32_t *slot_of(uint32_t *slots, int stage, int u) {
    return slots + ((size_t)(stage * GUNROLL + u) * GTHREADS + threadIdx.x) * VEC;
}

template <int VEC>
__device__ __forceinline__ Words<VEC> read_slot(const uint32_t *p) {
    using V = typename WordVec<VEC>::type;
    V v = *reinterpret_cast<const V *>(p);
    Words<VEC> out;
    memcpy(out.w, &v, sizeof(V));
    return out;
}

__host__ __device__ constexpr size_t slots_bytes(int vec) { return (size_t)STAGES * GUNROLL * GTHREADS * vec * 4; }

// ---------------------------------------------------------------- gather
// dst row = [coded row XOR] XOR over operands of the batch sums of a segment.
// Serves pre-combining (1 operand), encoding (r operands) and the stepwise
// decode (coded row and r-1 operands).  A batch sum adds the b files of a
// batch in ascending order starting from the first file's value (the
// pre-combined value of Section IV-B) and is zero where the segment does not
// exist.
struct GatherParams {
    const uint32_t *src[CCDC_MAX_K];
    uint32_t *dst[CCDC_MAX_K];
    const uint32_t *coded_in;
    const ccdc_row *rows;
    const ccdc_ref *refs;
    long long nrows;
    long long spans_per_row;
    long long span_elems;       // elements of a row one block covers (a multiple of the tile)
    long long file_stride;
    long long dst_add;          // added to every row's destination offset
    int na;
    int b;
    int replicas;               // > 0: every row is stored into dst[0..replicas-1] (peer buffers)
};

// position in a block's chunk sequence: for each tile of the span, the coded
// row (operand -1, if any), then operand a = 0..na-1, file f = 0..b-1
struct GatherCursor {
    long long base;
    int a, f;
};

template <int VEC, bool F32>
__global__ void __launch_bounds__(GTHREADS)
k_gather(const __grid_constant__ GatherParams p) {
    constexpr long long TILE = (long long)GTHREADS * VEC * GUNROLL;
    extern __shared__ __align__(16) uint32_t slots[];
    __shared__ ccdc_ref sh_refs[CCDC_MAX_K];
    const long long item = blockIdx.x;
    const long long row = item / p.spans_per_row;
    const long long span = item - row * p.spans_per_row;
    if (row >= p.nrows) return;
    const ccdc_row R = p.rows[row];
    const long long begin = span * p.span_elems;
    const long long end = min(R.n, begin + p.span_elems);
    if (begin >= end) return;
    pdl_trigger();
    if (threadIdx.x < p.na) sh_refs[threadIdx.x] = p.refs[row * p.na + threadIdx.x];
    __syncthreads();
    pdl_wait();
    const uint32_t *src = p.src[R.src_node];
    uint32_t *dst = p.dst[R.dst_node] + R.dst_off;
    const int a0 = R.coded_off >= 0 ? -1 : 0;
    const int nb = R.nf > 0 ? (int)R.nf : p.b;       // files summed per operand
    const long long tj = (long long)threadIdx.x * VEC;

    auto advance = [&](GatherCursor &c) {
        if (c.a >= 0 && ++c.f < nb) return;
        c.f = 0;
        if (++c.a >= p.na) { c.a = a0; c.base += TILE; }
    };
    // global address and validity of this thread's vector u of the chunk at c
    auto locate = [&](const GatherCursor &c, int u, const uint32_t *&g) -> bool {
        const long long j = c.base + tj + (long long)u * GTHREADS * VEC;
        if (c.a < 0) { g = p.coded_in + R.coded_off + j; return j < end; }
        const ccdc_ref E = sh_refs[c.a];
        g = src + E.off + c.f * p.file_stride + j;
        return j < end && j < E.vl;
    };
    auto issue = [&](const GatherCursor &c, int stage) {
#pragma unroll
        for (int u = 0; u < GUNROLL; ++u) {
            const uint32_t *g;
            if (locate(c, u, g)) async_copy<VEC>(slot_of<VEC>(slots, stage, u), g);
        }
    };

    GatherCursor ic{begin, a0, 0}, cc{begin, a0, 0};
    for (int i = 0; i < STAGES - 1; ++i) {
        if (ic.base < end) { issue(ic, i); advance(ic); }
        async_commit();
    }
    Words<VEC> x[GUNROLL], sum[GUNROLL];
#pragma unroll
    for (int u = 0; u < GUNROLL; ++u) x[u] = sum[u] = zero_words<VEC>();
    int stage = 0;
    while (cc.base < end) {
        if (ic.base < end) { issue(ic, stage == 0 ? STAGES - 1 : stage - 1); advance(ic); }
        async_commit();
        async_wait<STAGES - 1>();
        const bool last_file = cc.a < 0 || cc.f == nb - 1;
        const bool last_of_tile = last_file && cc.a == p.na - 1;
#pragma unroll
        for (int u = 0; u < GUNROLL; ++u) {
            const uint32_t *g;
            const bool ok = locate(cc, u, g);
            const Words<VEC> v = ok ? read_slot<VEC>(slot_of<VEC>(slots, stage, u)) : zero_words<VEC>();
            if (cc.a < 0) {
                x[u] = v;
            } else {
                if (cc.f == 0) sum[u] = v; else add_into<VEC, F32>(sum[u], v);
                if (last_file) xor_into<VEC>(x[u], sum[u]);
            }
            if (last_of_tile) {
                const long long j = cc.base + tj + (long long)u * GTHREADS * VEC;
                if (j < end) store_words<VEC>(dst + j, x[u]);
                x[u] = zero_words<VEC>();
            }
        }
        advance(cc);
        stage = stage + 1 == STAGES ? 0 : stage + 1;
    }
}

// Lean variant for the common shapes: RS operands known at compile time, no
// coded input.  The loads of G files of every operand (RS x G x SU vectors) are
// issued from registers before any is consumed; no shared memory, no barrier.
// A batch of more than G files takes further groups of G, added in file order.
#ifndef CCDC_STATIC_GATHER_THREADS
#define CCDC_STATIC_GATHER_THREADS 256
#endif
#ifndef CCDC_GATHER_WIDE_ROW
#define CCDC_GATHER_WIDE_ROW (1 << 15)    // one-file rows of at least this many words get blocks of twice the threads
#endif
#ifndef CCDC_GATHER_FILES_VECTORS
#define CCDC_GATHER_FILES_VECTORS 2       // vectors per thread per tile when several files are loaded together
#endif
#ifndef CCDC_GATHER_GROUP_WORDS
#define CCDC_GATHER_GROUP_WORDS 32        // most words per thread a group of files may keep in flight
#endif
#ifndef CCDC_GATHER_FILES_THREADS
#define CCDC_GATHER_FILES_THREADS 128     // threads per block when several files are loaded together
#endif
constexpr int STHREADS = CCDC_STATIC_GATHER_THREADS;
constexpr int FTHREADS = CCDC_GATHER_FILES_THREADS;
constexpr int FSU = CCDC_GATHER_FILES_VECTORS;

template <int VEC, bool F32, int RS, int G, int SU, int NT>
__global__ void __launch_bounds__(NT)
k_gather_static(const __grid_constant__ GatherParams p) {
    constexpr long long TILE = (long long)NT * VEC * SU;
    const long long item = blockIdx.x;
    if (item >= p.nrows * p.spans_per_row) return;
    // the dependent kernel may be scheduled, and this block's table entries fetched, while the previous
    // kernel of the stream drains; no data buffer is touched before pdl_wait
    pdl_trigger();
    const long long row = item / p.spans_per_row;
    const ccdc_row R = p.rows[row];
    ccdc_ref E[RS];
#pragma unroll
    for (int a = 0; a < RS; ++a) E[a] = p.refs[row * RS + a];
    pdl_wait();
    const long long span = item - row * p.spans_per_row;
    const long long begin = span * p.span_elems;
    const long long end = min(R.n, begin + p.span_elems);
    const int nb = G == 1 ? 1 : (R.nf > 0 ? (int)R.nf : p.b);      // files summed per operand
    const uint32_t *src = p.src[R.src_node];
    uint32_t *dst = p.dst[p.replicas > 0 ? 0 : R.dst_node] + R.dst_off + p.dst_add;
    for (long long base = begin; base < end; base += TILE) {
        Words<VEC> v[RS][SU];
        for (int f0 = 0; f0 < nb; f0 += G) {
            Words<VEC> w[G][RS][SU];
#pragma unroll
            for (int x = 0; x < G; ++x)
#pragma unroll
                for (int a = 0; a < RS; ++a)
#pragma unroll
                    for (int u = 0; u < SU; ++u) {
                        const long long j = base + ((long long)u * NT + threadIdx.x) * VEC;
                        w[x][a][u] = (f0 + x < nb && j < end && j < E[a].vl)
                                         ? load_words<VEC>(src + E[a].off + (f0 + x) * p.file_stride + j)
                                         : zero_words<VEC>();
                    }
#pragma unroll
            for (int x = 0; x < G; ++x) {
                if (f0 + x >= nb) break;
#pragma unroll
                for (int a = 0; a < RS; ++a)
#pragma unroll
                    for (int u = 0; u < SU; ++u) {
                        if (f0 + x == 0) v[a][u] = w[0][a][u];              // the sum starts from the first file's value
                        else add_into<VEC, F32>(v[a][u], w[x][a][u]);
                    }
            }
        }
#pragma unroll
        for (int u = 0; u < SU; ++u) {
            const long long j = base + ((long long)u * NT + threadIdx.x) * VEC;
#pragma unroll
            for (int a = 1; a < RS; ++a) xor_into<VEC>(v[0][u], v[a][u]);
            if (j < end) {
                store_words<VEC>(dst + j, v[0][u]);
                // the same row into every other peer's buffer (plain stores over NVLink when the
                // pointers are peer mappings): the all-gather happens as the rows are produced
                for (int d = 1; d < p.replicas; ++d)
                    store_words<VEC>(p.dst[d] + R.dst_off + p.dst_add + j, v[0][u]);
            }
        }
    }
}

// ------------------------------------------------------ fused decode + reduce
// One block: node k (row of outputs), one segment i, one tile of it, one chunk
// of the job's batches.  For each batch, ascending: the locally pre-combined
// value if k stores the batch, else the coded word XOR the r-1 cancellable
// pre-combined words (Section IV-B decoding), added to the accumulator
// (Eq. (1)).  Decoded packets never reach memory.
//
// When the batch loop is split over several blocks (chunks), every block
// leaves its partial sum in the workspace and k_sum_chunks adds them in chunk
// order.  (Letting the block that finishes a cell last add them inside this
// kernel was tried: no faster on any workload, and the extra code disturbed
// the register allocation of the streaming loop.)
struct DecodeParams {
    const uint32_t *part[CCDC_MAX_K];
    const uint32_t *coded;
    uint32_t *out;          // [out rows][len]
    uint32_t *ws;           // [nchunk][out rows][len] when nchunk > 1
    const ccdc_ref *terms;  // [out rows][r][nterm][TS]
    const int *out_rows;    // the out rows to compute (node-sharded plans), or NULL for all
    long long nlist;        // how many
    long long nout;         // out rows = J*K
    long long len, s;
    long long file_stride;
    long long tiles_per_seg;
    long long tile_span;    // consecutive tiles of a segment one block walks
    long long spans_per_seg;
    long long nterm, terms_per_chunk;
    int K, r, b, TS, nchunk;
    int stage_terms;        // terms staged in shared memory at a time
};

// R1S >= 0: r-1 = R1S is a compile-time constant and the loads of a batch --
// the coded word and G files of each of the r-1 operands, or G files of a
// local batch -- are issued together; batches of more than G files take
// further groups of G.  The loads of DEPTH consecutive batches are issued
// before any is consumed (about 64 KiB of loads in flight per SM is what the
// HBM read rate needs).  R1S < 0: any r, batch by batch.
// A block walks `tile_span` consecutive tiles of its segment; when its whole chunk of the term table
// fits the shared-memory stage it is staged once for all of them.
// Blocks per SM the register allocation is held to (the compiler's own choice moves with every
// change to the kernel, and the streaming rate follows the resident threads): blocks of 512 threads
// with little in flight per thread at 3 per SM (40 registers), with more at 2 (64); several files in
// flight: 6 blocks of 128 threads (80 registers) with 128-bit accesses, 7 (72 registers, which those
// kernels fill without spilling) with narrower ones.
constexpr int decode_min_blocks(int vec, int nt, int r1s, int g) {
    if (g > 1) return nt <= 128 ? CCDC_DECODE_BLOCKS_FILES(vec) : nt <= 256 ? 3 : 2;
    if (nt >= 1024) return 1;
    if (r1s < 0) return vec <= 2 ? 3 : 2;
    return (1 + r1s) * vec * CCDC_DECODE_DEPTH <= 16 ? 3 : 2;
}

// CL: the blocks that share an output tile (one per chunk of the split batch loop) form a thread-block
// cluster and add their partial sums through distributed shared memory, in chunk order, instead of
// through the workspace and a second launch.
template <int VEC, bool F32, int NT, int R1S, int G, bool CL>
__global__ void __launch_bounds__(NT, decode_min_blocks(VEC, NT, R1S, G))
k_decode_reduce(const __grid_constant__ DecodeParams p) {
    constexpr long long TILE = (long long)NT * VEC * DUNROLL;
    extern __shared__ ccdc_ref sh_terms[];

    long long item = blockIdx.x;
    int chunk = 0;
    if constexpr (CL) { chunk = (int)(item % p.nchunk); item /= p.nchunk; }     // the rank in the cluster
    const long long span = item % p.spans_per_seg; item /= p.spans_per_seg;
    const int i = (int)(item % p.r); item /= p.r;
    if constexpr (!CL) { chunk = (int)(item % p.nchunk); item /= p.nchunk; }
    const long long li = item;
    if (li >= p.nlist) return;
    const long long orow = p.out_rows ? p.out_rows[li] : li;

    const long long seglen = min(p.s, max(0LL, p.len - (long long)i * p.s));
    const int k = (int)(orow % p.K);
    const uint32_t *src = p.part[k];
    const int r1 = p.r - 1;

    const long long t_begin = (long long)chunk * p.terms_per_chunk;
    const long long t_end = min(p.nterm, t_begin + p.terms_per_chunk);
    const ccdc_ref *table = p.terms + ((orow * p.r + i) * p.nterm) * p.TS;
    // one-file batches: a block takes a single tile (SPAN false: no loop state in the streaming loop)
    constexpr bool SPAN = G > 1;
    const bool staged_once = SPAN && t_end - t_begin <= p.stage_terms;
    pdl_trigger();
    if (staged_once) {
        for (int x = threadIdx.x; x < (int)(t_end - t_begin) * p.TS; x += NT) sh_terms[x] = table[t_begin * p.TS + x];
        __syncthreads();
    }
    pdl_wait();

    const long long tile_first = SPAN ? span * p.tile_span : span;
    const long long tile_end = SPAN ? min(p.tiles_per_seg, (span + 1) * p.tile_span) : span + 1;
    for (long long tile = tile_first; tile < tile_end; ++tile) {
    if (tile * TILE >= seglen) break;
    const long long j0 = tile * TILE + (long long)threadIdx.x * VEC;
    Words<VEC> acc[DUNROLL];
#pragma unroll
    for (int u = 0; u < DUNROLL; ++u) acc[u] = zero_words<VEC>();

    for (long long t0 = t_begin; t0 < t_end; t0 += p.stage_terms) {
        const int nt = (int)min((long long)p.stage_terms, t_end - t0);
        if (!staged_once) {
            __syncthreads();
            for (int x = threadIdx.x; x < nt * p.TS; x += NT) sh_terms[x] = table[t0 * p.TS + x];
            __syncthreads();
        }
        if constexpr (R1S >= 0) {
            constexpr int NSLOT = (1 + R1S * G) > G ? (1 + R1S * G) : G;     // vectors a batch keeps in flight
            constexpr int DEPTH = NSLOT * VEC * DUNROLL <= CCDC_DECODE_DEPTH_WORDS ? (G > 1 ? CCDC_DECODE_DEPTH_FILES : CCDC_DECODE_DEPTH) : 1;
            const int nb = G == 1 ? 1 : p.b;
            for (int t = 0; t < nt; t += DEPTH) {
                Words<VEC> v[DEPTH][NSLOT][DUNROLL];
#pragma unroll
                for (int x = 0; x < DEPTH; ++x) {              // every first-group load of DEPTH batches first
                    if (t + x >= nt) break;
                    const ccdc_ref *e = sh_terms + (t + x) * p.TS;
                    const long long coded_off = e[0].off;
#pragma unroll
                    for (int u = 0; u < DUNROLL; ++u) {
                        const long long j = j0 + (long long)u * NT * VEC;
                        if (coded_off < 0) {
                            const uint32_t *q = src + e[1].off + j;
#pragma unroll
                            for (int f = 0; f < G; ++f)
                                v[x][f][u] = (f < nb && j < seglen) ? load_words<VEC>(q + f * p.file_stride) : zero_words<VEC>();
                        } else {
                            v[x][0][u] = j < seglen ? load_words<VEC>(p.coded + coded_off + j) : zero_words<VEC>();
#pragma unroll
                            for (int c = 1; c <= R1S; ++c) {
                                const uint32_t *q = src + e[c].off + j;
                                const bool ok = j < seglen && j < e[c].vl;
#pragma unroll
                                for (int f = 0; f < G; ++f)
                                    v[x][1 + (c - 1) * G + f][u] = (f < nb && ok) ? load_words<VEC>(q + f * p.file_stride)
                                                                                  : zero_words<VEC>();
                            }
                        }
                    }
                }
#pragma unroll
                for (int x = 0; x < DEPTH; ++x) {              // then consume them in batch order
                    if (t + x >= nt) break;
                    const ccdc_ref *e = sh_terms + (t + x) * p.TS;
                    const bool local = e[0].off < 0;
#pragma unroll
                    for (int u = 0; u < DUNROLL; ++u) {
                        const long long j = j0 + (long long)u * NT * VEC;
                        // sum over the files of one operand whose first group sits in slots first..first+G-1
                        auto operand = [&](int first, const ccdc_ref E, long long vl) -> Words<VEC> {
                            Words<VEC> sum = v[x][first][u];
#pragma unroll
                            for (int f = 1; f < G; ++f)
                                if (f < nb) add_into<VEC, F32>(sum, v[x][first + f][u]);
                            for (int f0 = G; f0 < nb; f0 += G) {            // batches of more than G files
                                Words<VEC> w[G];
#pragma unroll
                                for (int f = 0; f < G; ++f)
                                    w[f] = (f0 + f < nb && j < vl) ? load_words<VEC>(src + E.off + j + (f0 + f) * p.file_stride)
                                                                   : zero_words<VEC>();
#pragma unroll
                                for (int f = 0; f < G; ++f)
                                    if (f0 + f < nb) add_into<VEC, F32>(sum, w[f]);
                            }
                            return sum;
                        };
                        Words<VEC> val;
                        if (local) {
                            val = operand(0, e[1], seglen);
                        } else {
                            val = v[x][0][u];
#pragma unroll
                            for (int c = 1; c <= R1S; ++c)
                                xor_into<VEC>(val, operand(1 + (c - 1) * G, e[c], min(seglen, e[c].vl)));
                        }
                        add_into<VEC, F32>(acc[u], val);
                    }
                }
            }
        } else {
            for (int t = 0; t < nt; ++t) {
                const ccdc_ref *e = sh_terms + t * p.TS;
                const long long coded_off = e[0].off;
                Words<VEC> v[DUNROLL];
                if (coded_off < 0) {
                    const ccdc_ref E = e[1];
#pragma unroll
                    for (int u = 0; u < DUNROLL; ++u) {
                        const long long j = j0 + (long long)u * NT * VEC;
                        v[u] = batch_sum<VEC, F32>(src, E.off, j, seglen, p.b, p.file_stride);
                    }
                } else {
#pragma unroll
                    for (int u = 0; u < DUNROLL; ++u) {
                        const long long j = j0 + (long long)u * NT * VEC;
                        v[u] = j < seglen ? load_words<VEC>(p.coded + coded_off + j) : zero_words<VEC>();
                    }
                    for (int c = 1; c <= r1; ++c) {
                        const ccdc_ref E = e[c];
#pragma unroll
                        for (int u = 0; u < DUNROLL; ++u) {
                            const long long j = j0 + (long long)u * NT * VEC;
                            if (j < seglen)
                                xor_into<VEC>(v[u], batch_sum<VEC, F32>(src, E.off, j, E.vl, p.b, p.file_stride));
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < DUNROLL; ++u) add_into<VEC, F32>(acc[u], v[u]);
            }
        }
    }
    const long long cell_off = orow * p.len + (long long)i * p.s;
    if constexpr (CL) {
        // every block of the cluster reaches this point for the same tiles (same segment, same span)
        __shared__ __align__(16) uint32_t sh_part[NT * VEC * DUNROLL];
#pragma unroll
        for (int u = 0; u < DUNROLL; ++u) store_words<VEC>(sh_part + (u * NT + (int)threadIdx.x) * VEC, acc[u]);
        cluster_sync();
        if (chunk == 0) {
            for (int c = 1; c < p.nchunk; ++c) {
#pragma unroll
                for (int u = 0; u < DUNROLL; ++u)
                    add_into<VEC, F32>(acc[u], load_words_peer<VEC>(sh_part + (u * NT + (int)threadIdx.x) * VEC, (unsigned)c));
            }
#pragma unroll
            for (int u = 0; u < DUNROLL; ++u) {
                const long long j = j0 + (long long)u * NT * VEC;
                if (j < seglen) store_words<VEC>(p.out + cell_off + j, acc[u]);
            }
        }
        cluster_sync();         // a peer's shared memory stays as it is until rank 0 has read it
        continue;
    }
    // the output, or this chunk's partial sum when the batch loop is split
    uint32_t *dst = (p.nchunk == 1 ? p.out : p.ws + (long long)chunk * p.nout * p.len) + cell_off;
#pragma unroll
    for (int u = 0; u < DUNROLL; ++u) {
        const long long j = j0 + (long long)u * NT * VEC;
        if (j < seglen) store_words<VEC>(dst + j, acc[u]);
    }
    }   // tiles of the span
}

// final pass of a split batch loop when the decode kernel leaves the partial sums in the workspace:
// out = ((ws[0] + ws[1]) + ...) in chunk order
template <bool F32>
__global__ void __launch_bounds__(DTHREADS)
k_sum_chunks(const uint32_t *__restrict__ ws, uint32_t *__restrict__ out, const int *__restrict__ out_rows,
             long long nlist, long long len, long long n, int nchunk) {
    const long long x = (long long)blockIdx.x * DTHREADS + threadIdx.x;
    if (x >= nlist * len) return;
    const long long li = x / len;
    const long long e = (out_rows ? out_rows[li] : li) * len + (x - li * len);
    pdl_trigger();
    pdl_wait();
    uint32_t acc = ws[e];
    for (int c = 1; c < nchunk; c += 8) {           // eight chunks' loads in flight, added in chunk order
        uint32_t w[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) w[x] = c + x < nchunk ? ws[(long long)(c + x) * n + e] : 0u;
#pragma unroll
        for (int x = 0; x < 8; ++x)
            if (c + x < nchunk) acc = add_word<F32>(acc, w[x]);
    }
    out[e] = acc;
}

// ------------------------------------------------------ stepwise reduce
// out row of node k = sum over the job's batches, ascending, of the local
// pre-combined value or the decoded packet (Eq. (1)).
struct ReduceParams {
    const uint32_t *part[CCDC_MAX_K];
    const uint32_t *decoded[CCDC_MAX_K];
    uint32_t *out;
    const ccdc_ref *terms;  // [out rows][nterm]
    long long nout, len, nterm, file_stride, tiles_per_row;
    int K, b;
};

template <int VEC, bool F32>
__global__ void __launch_bounds__(DTHREADS, 2)      // two blocks per SM: up to 64 registers
k_reduce(const __grid_constant__ ReduceParams p) {
    constexpr long long TILE = (long long)DTHREADS * VEC;
    const long long orow = blockIdx.x / p.tiles_per_row;
    const long long tile = blockIdx.x - orow * p.tiles_per_row;
    if (orow >= p.nout) return;
    const long long j = tile * TILE + (long long)threadIdx.x * VEC;
    if (j >= p.len) return;
    const int k = (int)(orow % p.K);
    const ccdc_ref *terms = p.terms + orow * p.nterm;
    pdl_trigger();
    pdl_wait();
    Words<VEC> acc = zero_words<VEC>();
    for (long long t = 0; t < p.nterm; t += 4) {            // four batches' loads in flight, added in batch order
        Words<VEC> v[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            if (t + x >= p.nterm) break;
            const ccdc_ref E = terms[t + x];
            v[x] = E.vl <= 0 ? batch_sum<VEC, F32>(p.part[k], E.off, j, p.len, E.vl < 0 ? (int)-E.vl : p.b, p.file_stride)
                             : load_words<VEC>(p.decoded[k] + E.off + j);
        }
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            if (t + x >= p.nterm) break;
            add_into<VEC, F32>(acc, v[x]);
        }
    }
    store_words<VEC>(p.out + orow * p.len + j, acc);
}

// ---------------------------------------------------------------- launching
template <typename F>
int dispatch(const ccdc_plan_s &P, F &&f) {
    const bool f32 = P.dtype == CCDC_F32;
    switch (P.vec) {
    case 4: return f32 ? f(std::integral_constant<int, 4>(), std::true_type()) : f(std::integral_constant<int, 4>(), std::false_type());
    case 2: return f32 ? f(std::integral_constant<int, 2>(), std::true_type()) : f(std::integral_constant<int, 2>(), std::false_type());
    default: return f32 ? f(std::integral_constant<int, 1>(), std::true_type()) : f(std::integral_constant<int, 1>(), std::false_type());
    }
}

int check_launch() {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? CCDC_OK : cuda_fail(e);
}

// kernels that stage more than the default 48 KiB of dynamic shared memory
// must opt in (a function attribute; nothing is allocated)
template <typename Kernel>
int allow_shared_memory(Kernel kernel, size_t bytes) {
    if (bytes <= 32 * 1024) return CCDC_OK;         // static shared memory shares the 48 KiB default
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    return e == cudaSuccess ? CCDC_OK : cuda_fail(e);
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_ptr_array(const ccdc_plan_s &P, const void *const *a, bool (*nonempty)(const ccdc_plan_s &, int)) {
    if (!a) return CCDC_EINVAL;
    for (int k = 0; k < P.K; ++k) {
        if (!nonempty(P, k)) continue;
        if (!a[k] || !aligned16(a[k])) return CCDC_EINVAL;
    }
    return CCDC_OK;
}

bool is_local(const ccdc_plan_s &P, int k) { return k / (P.K / P.shard_world) == P.shard_rank; }
bool has_part(const ccdc_plan_s &P, int k) { return P.nlocal[k] > 0 && is_local(P, k); }
bool has_decoded(const ccdc_plan_s &P, int k) { return P.node_nrounds[k] > 0 && is_local(P, k); }

int launch_gather(const ccdc_plan_s &P, const ccdc_gather_table &T, const void *const *src, void *const *dst,
                  void *dst_single, const void *coded_in, int b, long long file_stride, cudaStream_t st,
                  void *const *peers = nullptr, int npeers = 0, long long dst_add = 0) {
    if (T.rows.empty() || T.n_max == 0) return CCDC_OK;
    GatherParams gp;
    std::memset(&gp, 0, sizeof(gp));
    for (int k = 0; k < P.K; ++k) {
        gp.src[k] = static_cast<const uint32_t *>(src[k]);
        gp.dst[k] = static_cast<uint32_t *>(dst_single ? dst_single : dst[k]);
    }
    if (npeers > 0) {
        for (int d = 0; d < npeers; ++d) gp.dst[d] = static_cast<uint32_t *>(peers[d]);
        gp.replicas = npeers;
        gp.dst_add = dst_add;
    }
    gp.coded_in = static_cast<const uint32_t *>(coded_in);
    gp.rows = T.d_rows; gp.refs = T.d_refs;
    gp.nrows = (long long)T.rows.size();
    gp.file_stride = file_stride; gp.na = T.na; gp.b = b;
    return dispatch(P, [&](auto vec, auto f32) -> int {
        constexpr int VEC = decltype(vec)::value;
        constexpr bool F32 = decltype(f32)::value;
        const bool lean = !coded_in && T.na >= 1 && T.na <= 4;
        if (npeers > 0 && !lean) return CCDC_ESIZE;         // peer stores exist in the lean kernel only
        const long long bmax = T.uniform ? b : T.nf_max;    // most files summed per operand
        // files whose loads are issued together: all of a small batch, fewer while the registers
        // of a thread would have to hold more than 48 words of them
        int group = bmax <= 1 ? 1 : bmax == 2 ? 2 : 4;
        while (group > 2 && T.na * group * VEC * FSU > CCDC_GATHER_GROUP_WORDS) group /= 2;
        // long one-file rows (the gradient-sized workload): 512-thread blocks measured 2 % faster; short rows lose with them
        const bool wide = lean && group == 1 && T.n_max >= (long long)CCDC_GATHER_WIDE_ROW;
        const int sthreads = wide ? 2 * STHREADS : group > 1 ? FTHREADS : STHREADS;
        const int svectors = group == 1 ? 2 : FSU;          // vectors per thread per tile
        const long long tile = lean ? (long long)sthreads * VEC * svectors : (long long)GTHREADS * VEC * GUNROLL;
        // a block covers up to 32 tiles of a row, fewer while that would
        // leave the grid short of 16 blocks per SM
        long long tiles = 32;
        while (tiles > 1 && gp.nrows * ((T.n_max + tile * tiles - 1) / (tile * tiles)) < (long long)P.sm_count * 16) tiles /= 2;
        gp.span_elems = tile * tiles;
        gp.spans_per_row = (T.n_max + gp.span_elems - 1) / gp.span_elems;
        const long long blocks = gp.nrows * gp.spans_per_row;
        if (blocks > 0x7fffffffLL) return CCDC_ESIZE;
        if (lean) {
            auto go = [&](auto rs) {
                constexpr int RS = decltype(rs)::value;
                if (wide) launch_kernel(k_gather_static<VEC, F32, RS, 1, 2, 2 * STHREADS>, blocks, 2 * STHREADS, 0, st, gp);
                else if (group == 1) launch_kernel(k_gather_static<VEC, F32, RS, 1, 2, STHREADS>, blocks, STHREADS, 0, st, gp);
                else if (group == 2) launch_kernel(k_gather_static<VEC, F32, RS, 2, FSU, FTHREADS>, blocks, FTHREADS, 0, st, gp);
                else launch_kernel(k_gather_static<VEC, F32, RS, 4, FSU, FTHREADS>, blocks, FTHREADS, 0, st, gp);
            };
            switch (T.na) {
            case 1: go(std::integral_constant<int, 1>()); break;
            case 2: go(std::integral_constant<int, 2>()); break;
            case 3: go(std::integral_constant<int, 3>()); break;
            default: go(std::integral_constant<int, 4>()); break;
            }
            std::snprintf(g_last_gather, sizeof(g_last_gather), "k_gather_static<vec=%d,operands=%d,files=%d,vectors=%d,threads=%d>",
                          VEC, T.na, group, svectors, sthreads);
            return check_launch();
        }
        const size_t smem = slots_bytes(VEC);
        int rc = allow_shared_memory(k_gather<VEC, F32>, smem);
        if (rc != CCDC_OK) return rc;
        launch_kernel(k_gather<VEC, F32>, blocks, GTHREADS, smem, st, gp);
        std::snprintf(g_last_gather, sizeof(g_last_gather), "k_gather<vec=%d,threads=%d>", VEC, GTHREADS);
        return check_launch();
    });
}

int ensure_device(ccdc_plan_s *plan) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (plan->device == dev) return CCDC_OK;
    if (plan->device != -1) return CCDC_ESTATE;     // tables live on another device
    return ccdc_plan_upload(plan);
}

}  // namespace

int ccdc_internal_cuda_fail(int cuda_error) { return cuda_fail((cudaError_t)cuda_error); }
void ccdc_internal_count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

void ccdc_internal_release_device(ccdc_plan_s *plan) {
    if (plan->d_blob) {
        int cur = -1;
        cudaGetDevice(&cur);
        if (cur != plan->device) cudaSetDevice(plan->device);
        cudaFree(plan->d_blob);
        if (cur != plan->device && cur >= 0) cudaSetDevice(cur);
    }
    plan->d_blob = nullptr;
    plan->device = -1;
}

extern "C" {

int ccdc_last_cuda_error(void) { return g_last_cuda_error; }
const char *ccdc_last_gather_kernel(void) { return g_last_gather; }
const char *ccdc_last_decode_kernel(void) { return g_last_decode; }
int ccdc_num_kernel_launches(void) { return g_launches.load(); }

int ccdc_plan_upload(ccdc_plan_t *plan) {
    if (!plan) return CCDC_EINVAL;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (plan->device == dev) return CCDC_OK;
    if (plan->device != -1) return CCDC_ESTATE;
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_fail(e);
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail(e);
    plan->device_has_bulk_copies = major >= 9;
    if (major < 9) plan->decode_cluster = false;            // no thread-block clusters: the workspace path
    if (plan->family == 1 && !ccdc_stream_supported(*plan)) {      // a device without bulk copies
        plan->family = 0;
        ccdc_internal_choose_split(plan);
    }
    ccdc_internal_resplit(plan, sms);       // launch shapes for this device's SM count
    struct Piece { const void *src; size_t bytes; const void **dst; };
    ccdc_gather_table *tabs[4] = {&plan->enc_fused, &plan->cmb, &plan->enc_pk, &plan->dec_pk};
    Piece pieces[18];
    int np = 0;
    for (ccdc_gather_table *T : tabs) {
        pieces[np++] = {T->rows.data(), T->rows.size() * sizeof(ccdc_row), (const void **)&T->d_rows};
        pieces[np++] = {T->refs.data(), T->refs.size() * sizeof(ccdc_ref), (const void **)&T->d_refs};
    }
    pieces[np++] = {plan->dec_terms.data(), plan->dec_terms.size() * sizeof(ccdc_ref), (const void **)&plan->d_dec_terms};
    pieces[np++] = {plan->red_terms.data(), plan->red_terms.size() * sizeof(ccdc_ref), (const void **)&plan->d_red_terms};
    pieces[np++] = {plan->out_rows.data(), plan->out_rows.size() * sizeof(int), (const void **)&plan->d_out_rows};
    if (plan->family == 1) {                    // the row lists of the bulk-copy pipeline, for the final split
        ccdc_internal_build_stream_tables(plan);
        for (ccdc_stream_table *S : {&plan->dec_stream, &plan->enc_stream}) {
            pieces[np++] = {S->rows.data(), S->rows.size() * sizeof(ccdc_stream_row), (const void **)&S->d_rows};
            pieces[np++] = {S->cells.data(), S->cells.size() * sizeof(ccdc_stream_cell), (const void **)&S->d_cells};
            pieces[np++] = {S->chunk_row0.data(), S->chunk_row0.size() * sizeof(int), (const void **)&S->d_chunk_row0};
        }
    }
    static const int zero_status = 0;           // the word a kernel sets when a bounded wait runs out
    pieces[np++] = {&zero_status, sizeof(int), (const void **)&plan->d_status};
    size_t total = 0;
    for (int i = 0; i < np; ++i) total += (pieces[i].bytes + 255) / 256 * 256;
    void *blob = nullptr;
    e = cudaMalloc(&blob, total ? total : 256);
    if (e != cudaSuccess) { g_last_cuda_error = (int)e; return e == cudaErrorMemoryAllocation ? CCDC_ENOMEM : CCDC_ECUDA; }
    size_t at = 0;
    for (int i = 0; i < np; ++i) {
        char *d = static_cast<char *>(blob) + at;
        if (pieces[i].bytes) {
            e = cudaMemcpy(d, pieces[i].src, pieces[i].bytes, cudaMemcpyHostToDevice);
            if (e != cudaSuccess) { cudaFree(blob); return cuda_fail(e); }
        }
        *pieces[i].dst = d;
        at += (pieces[i].bytes + 255) / 256 * 256;
    }
    plan->d_blob = blob;
    plan->device = dev;
    return CCDC_OK;
}

int ccdc_combine(ccdc_plan_t *plan, const void *const *part, void *const *packets, void *stream) {
    if (plan && plan->shard_world > 1) return CCDC_ESTATE;       // the stepwise API is single-GPU
    if (plan && plan->compression_mode) return CCDC_ESTATE;     // no coded path in a compression-only plan
    if (!plan) return CCDC_EINVAL;
    int rc = check_ptr_array(*plan, part, has_part);
    if (rc == CCDC_OK) rc = check_ptr_array(*plan, (const void *const *)packets, has_part);
    if (rc == CCDC_OK) rc = ensure_device(plan);
    if (rc != CCDC_OK) return rc;
    return launch_gather(*plan, plan->cmb, part, packets, nullptr, nullptr, (int)plan->b, plan->row_elems,
                         static_cast<cudaStream_t>(stream));
}

int ccdc_encode(ccdc_plan_t *plan, const void *const *packets, void *coded, void *stream) {
    if (plan && plan->shard_world > 1) return CCDC_ESTATE;       // the stepwise API is single-GPU
    if (plan && plan->compression_mode) return CCDC_ESTATE;     // no coded path in a compression-only plan
    if (!plan || !coded || !aligned16(coded)) return CCDC_EINVAL;
    int rc = check_ptr_array(*plan, packets, has_part);
    if (rc == CCDC_OK) rc = ensure_device(plan);
    if (rc != CCDC_OK) return rc;
    return launch_gather(*plan, plan->enc_pk, packets, nullptr, coded, nullptr, 1, 0,
                         static_cast<cudaStream_t>(stream));
}

int ccdc_decode(ccdc_plan_t *plan, const void *const *packets, const void *coded, void *const *decoded,
                void *stream) {
    if (plan && plan->shard_world > 1) return CCDC_ESTATE;       // the stepwise API is single-GPU
    if (plan && plan->compression_mode) return CCDC_ESTATE;     // no coded path in a compression-only plan
    if (!plan || !coded || !aligned16(coded)) return CCDC_EINVAL;
    int rc = check_ptr_array(*plan, packets, has_part);
    if (rc == CCDC_OK) rc = check_ptr_array(*plan, (const void *const *)decoded, has_decoded);
    if (rc == CCDC_OK) rc = ensure_device(plan);
    if (rc != CCDC_OK) return rc;
    return launch_gather(*plan, plan->dec_pk, packets, decoded, nullptr, coded, 1, 0,
                         static_cast<cudaStream_t>(stream));
}

int ccdc_reduce(ccdc_plan_t *plan, const void *const *part, const void *const *decoded, void *out, void *stream) {
    if (plan && plan->shard_world > 1) return CCDC_ESTATE;       // the stepwise API is single-GPU
    if (!plan || !out || !aligned16(out)) return CCDC_EINVAL;
    int rc = check_ptr_array(*plan, part, has_part);
    if (rc == CCDC_OK) rc = check_ptr_array(*plan, decoded, has_decoded);
    if (rc == CCDC_OK) rc = ensure_device(plan);
    if (rc != CCDC_OK) return rc;
    const ccdc_plan_s &P = *plan;
    ReduceParams rp;
    std::memset(&rp, 0, sizeof(rp));
    for (int k = 0; k < P.K; ++k) {
        rp.part[k] = static_cast<const uint32_t *>(part[k]);
        rp.decoded[k] = static_cast<const uint32_t *>(decoded[k]);
    }
    rp.out = static_cast<uint32_t *>(out);
    rp.terms = P.d_red_terms;
    rp.nout = P.J * P.K; rp.len = P.len; rp.nterm = P.nterm; rp.file_stride = P.row_elems;
    rp.K = P.K; rp.b = (int)P.b;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return dispatch(P, [&](auto vec, auto f32) -> int {
        constexpr int VEC = decltype(vec)::value;
        constexpr bool F32 = decltype(f32)::value;
        const long long tile = (long long)DTHREADS * VEC;
        rp.tiles_per_row = (P.len + tile - 1) / tile;
        const long long blocks = rp.nout * rp.tiles_per_row;
        if (blocks > 0x7fffffffLL) return CCDC_ESIZE;
        launch_kernel(k_reduce<VEC, F32>, blocks, DTHREADS, 0, st, rp);
        return check_launch();
    });
}

int ccdc_encode_fused(ccdc_plan_t *plan, const void *const *part, void *coded, void *stream) {
    if (plan && plan->compression_mode) return CCDC_ESTATE;     // no coded path in a compression-only plan
    if (!plan || !coded || !aligned16(coded)) return CCDC_EINVAL;
    int rc = check_ptr_array(*plan, part, has_part);
    if (rc == CCDC_OK) rc = ensure_device(plan);
    if (rc != CCDC_OK) return rc;
    if (plan->family == 1) {
        std::snprintf(g_last_gather, sizeof(g_last_gather), "k_stream<encode,tile=%lld>", ccdc_stream_tile_words());
        return ccdc_stream_encode(*plan, part, coded, static_cast<cudaStream_t>(stream));
    }
    return launch_gather(*plan, plan->enc_fused, part, nullptr, coded, nullptr, (int)plan->b, plan->row_elems,
                         static_cast<cudaStream_t>(stream));
}

int ccdc_encode_fused_peers(ccdc_plan_t *plan, const void *const *part, void *const *peer_coded, void *stream) {
    if (!plan || !peer_coded) return CCDC_EINVAL;
    if (plan->compression_mode || plan->shard_world < 2) return CCDC_ESTATE;
    if (plan->shard_world > CCDC_MAX_K) return CCDC_ESIZE;
    for (int d = 0; d < plan->shard_world; ++d)
        if (!peer_coded[d] || !aligned16(peer_coded[d])) return CCDC_EINVAL;
    int rc = check_ptr_array(*plan, part, has_part);
    if (rc == CCDC_OK) rc = ensure_device(plan);
    if (rc != CCDC_OK) return rc;
    // this rank's rows go to their gathered position in every rank's buffer
    return launch_gather(*plan, plan->enc_fused, part, nullptr, peer_coded[0], nullptr, (int)plan->b, plan->row_elems,
                         static_cast<cudaStream_t>(stream), peer_coded, plan->shard_world,
                         (long long)plan->shard_rank * plan->send_rows * plan->s_pad);
}

int ccdc_decode_reduce(ccdc_plan_t *plan, const void *const *part, const void *coded, void *out,
                       void *workspace, void *stream) {
    if (plan && plan->compression_mode) return CCDC_ESTATE;     // no coded path in a compression-only plan
    if (!plan || !coded || !out || !aligned16(coded) || !aligned16(out)) return CCDC_EINVAL;
    if (ccdc_workspace_bytes(plan) > 0 && (!workspace || !aligned16(workspace))) return CCDC_EINVAL;
    int rc = check_ptr_array(*plan, part, has_part);
    if (rc == CCDC_OK) rc = ensure_device(plan);
    if (rc != CCDC_OK) return rc;
    if (ccdc_workspace_bytes(plan) > 0 && !workspace) return CCDC_EINVAL;      // the upload may have re-sized the split
    const ccdc_plan_s &P = *plan;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DecodeParams dp;
    std::memset(&dp, 0, sizeof(dp));
    for (int k = 0; k < P.K; ++k) dp.part[k] = static_cast<const uint32_t *>(part[k]);
    dp.coded = static_cast<const uint32_t *>(coded);
    dp.out = static_cast<uint32_t *>(out);
    dp.ws = static_cast<uint32_t *>(workspace);
    dp.terms = P.d_dec_terms;
    dp.nout = P.J * P.K; dp.len = P.len; dp.s = P.s; dp.file_stride = P.row_elems;
    dp.out_rows = P.shard_world > 1 ? P.d_out_rows : nullptr;
    dp.nlist = P.shard_world > 1 ? (long long)P.out_rows.size() : dp.nout;
    dp.nterm = P.nterm; dp.terms_per_chunk = P.terms_per_chunk;
    dp.K = P.K; dp.r = P.r; dp.b = (int)P.b; dp.TS = P.term_stride; dp.nchunk = P.nchunk;
    if (P.family == 1) {
        std::snprintf(g_last_decode, sizeof(g_last_decode), "k_stream<decode,tile=%lld,chunks=%d>", ccdc_stream_tile_words(),
                      P.nchunk);
        rc = ccdc_stream_decode(P, part, coded, out, workspace, st);
        if (rc != CCDC_OK || P.nchunk == 1) return rc;
        const long long n = P.J * P.K * P.len;
        const long long todo = (P.shard_world > 1 ? (long long)P.out_rows.size() : P.J * P.K) * P.len;
        if (P.dtype == CCDC_F32)
            launch_kernel(k_sum_chunks<true>, (todo + DTHREADS - 1) / DTHREADS, DTHREADS, 0, st, (const uint32_t *)workspace,
                          static_cast<uint32_t *>(out), P.shard_world > 1 ? P.d_out_rows : (const int *)nullptr,
                          P.shard_world > 1 ? (long long)P.out_rows.size() : P.J * P.K, P.len, n, P.nchunk);
        else
            launch_kernel(k_sum_chunks<false>, (todo + DTHREADS - 1) / DTHREADS, DTHREADS, 0, st, (const uint32_t *)workspace,
                          static_cast<uint32_t *>(out), P.shard_world > 1 ? P.d_out_rows : (const int *)nullptr,
                          P.shard_world > 1 ? (long long)P.out_rows.size() : P.J * P.K, P.len, n, P.nchunk);
        return check_launch();
    }
    const int stage_refs = 1024;                                    // 16 KiB of shared memory
    dp.stage_terms = (int)std::max(1LL, std::min<long long>(stage_refs / P.term_stride, P.terms_per_chunk));
    return dispatch(P, [&](auto vec, auto f32) -> int {
        constexpr int VEC = decltype(vec)::value;
        constexpr bool F32 = decltype(f32)::value;
        const long long tile = (long long)P.decode_threads * VEC * DUNROLL;
        dp.tiles_per_seg = (P.s + tile - 1) / tile;
        // a block walks several tiles of its segment while the grid keeps 16 blocks per SM (amortises
        // the staging of a short term table: many jobs with few batches each)
        dp.tile_span = 1;
        while (P.decode_files > 1 && P.terms_per_chunk <= dp.stage_terms && P.terms_per_chunk <= 16 &&
               dp.tile_span < dp.tiles_per_seg && dp.tile_span < 8 &&
               dp.nlist * P.nchunk * P.r * ((dp.tiles_per_seg + 2 * dp.tile_span - 1) / (2 * dp.tile_span)) >= (long long)P.sm_count * 16)
            dp.tile_span *= 2;
        dp.spans_per_seg = (dp.tiles_per_seg + dp.tile_span - 1) / dp.tile_span;
        const long long blocks = dp.nlist * P.nchunk * P.r * dp.spans_per_seg;
        if (blocks > 0x7fffffffLL) return CCDC_ESIZE;
        const size_t smem = (size_t)dp.stage_terms * P.term_stride * sizeof(ccdc_ref);
        // small r and 64- or 128-bit accesses: the instantiation with r-1 and the files loaded together
        // as compile-time constants; everything else batch by batch
        const int group = P.decode_files;
        const bool fast = P.decode_files >= 1;
        const int r1s = fast ? P.r - 1 : -1;
        auto launch = [&](auto nt, auto r1, auto g) {
            constexpr int NT = decltype(nt)::value;
            constexpr int R1 = decltype(r1)::value;
            constexpr int G = decltype(g)::value;
            if constexpr (G > 1) {
                if (P.decode_cluster) {
                    launch_clustered(k_decode_reduce<VEC, F32, NT, R1, G, true>, P.nchunk, blocks, NT, smem, st, dp);
                    return;
                }
            }
            launch_kernel(k_decode_reduce<VEC, F32, NT, R1, G, false>, blocks, NT, smem, st, dp);
        };
        auto with_shape = [&](auto r1) {
            constexpr int R1 = decltype(r1)::value;
            constexpr bool GENERIC = R1 < 0;
            const int nt = P.decode_threads;
            if (!GENERIC && group == 4) launch(std::integral_constant<int, CCDC_DECODE_THREADS_FILES>(), r1, std::integral_constant<int, 4>());
            else if (!GENERIC && group == 2) launch(std::integral_constant<int, CCDC_DECODE_THREADS_FILES>(), r1, std::integral_constant<int, 2>());
            else if (nt == CCDC_DECODE_THREADS_SHORT) launch(std::integral_constant<int, CCDC_DECODE_THREADS_SHORT>(), r1, std::integral_constant<int, 1>());
            else launch(std::integral_constant<int, DTHREADS>(), r1, std::integral_constant<int, 1>());
        };
        if constexpr (VEC >= 2) {
            switch (r1s) {
            case 0: with_shape(std::integral_constant<int, 0>()); break;
            case 1: with_shape(std::integral_constant<int, 1>()); break;
            case 2: with_shape(std::integral_constant<int, 2>()); break;
            case 3: with_shape(std::integral_constant<int, 3>()); break;
            default: with_shape(std::integral_constant<int, -1>()); break;
            }
        } else {
            with_shape(std::integral_constant<int, -1>());
        }
        std::snprintf(g_last_decode, sizeof(g_last_decode), "k_decode_reduce<vec=%d,threads=%d,cancel=%d,files=%d,chunks=%d%s>",
                      VEC, P.decode_threads, r1s, group, P.nchunk, P.decode_cluster ? ",cluster" : "");
        int lrc = check_launch();
        if (lrc != CCDC_OK || P.nchunk == 1 || P.decode_cluster) return lrc;
        const long long n = dp.nout * P.len, todo = dp.nlist * P.len;
        launch_kernel(k_sum_chunks<F32>, (todo + DTHREADS - 1) / DTHREADS, DTHREADS, 0, st,
               (const uint32_t *)dp.ws, dp.out, dp.out_rows, dp.nlist, P.len, n, P.nchunk);
        return check_launch();
    });
}

int ccdc_shuffle_status(const ccdc_plan_t *plan) {
    if (!plan) return CCDC_EINVAL;
    if (!plan->d_status) return CCDC_OK;            // nothing has run yet
    int word = 0;
    const cudaError_t e = cudaMemcpy(&word, plan->d_status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e);
    return word == 0 ? CCDC_OK : CCDC_ESTATE;
}

int ccdc_shuffle(ccdc_plan_t *plan, const void *const *part, void *coded, void *out, void *workspace,
                 void *stream) {
    if (plan && plan->shard_world > 1) return CCDC_ESTATE;       // the coded rows must be exchanged between the two launches
    if (!plan || !coded || !out || !aligned16(coded) || !aligned16(out)) return CCDC_EINVAL;
    if (ccdc_workspace_bytes(plan) > 0 && (!workspace || !aligned16(workspace))) return CCDC_EINVAL;
    int rc = ccdc_encode_fused(plan, part, coded, stream);
    if (rc != CCDC_OK) return rc;
    return ccdc_decode_reduce(plan, part, coded, out, workspace, stream);
}

int ccdc_compression_shuffle(ccdc_plan_t *plan, const void *const *part, void *const *recv, void *out,
                             void *stream) {
    if (!plan || !out || !aligned16(out)) return CCDC_EINVAL;
    if (!plan->compression_mode) return CCDC_ESTATE;
    int rc = check_ptr_array(*plan, part, has_part);
    if (rc == CCDC_OK) rc = check_ptr_array(*plan, (const void *const *)recv, has_decoded);
    if (rc == CCDC_OK) rc = ensure_device(plan);
    if (rc != CCDC_OK) return rc;
    // unicast: the sender's pre-combined packet lands in the receiver's buffer
    rc = launch_gather(*plan, plan->cmb, part, recv, nullptr, nullptr, (int)plan->b, plan->row_elems,
                       static_cast<cudaStream_t>(stream));
    if (rc != CCDC_OK) return rc;
    return ccdc_reduce(plan, part, (const void *const *)recv, out, stream);
}

int ccdc_shuffle_host(ccdc_plan_t *plan, const void *const *host_part, void *host_out, void *const *dev_part,
                      void *dev_coded, void *dev_out, void *dev_workspace, void *stream) {
    if (!plan || !host_part || !host_out || !dev_part || !dev_coded || !dev_out) return CCDC_EINVAL;
    if (!aligned16(dev_coded) || !aligned16(dev_out)) return CCDC_EINVAL;
    if (ccdc_workspace_bytes(plan) > 0 && (!dev_workspace || !aligned16(dev_workspace))) return CCDC_EINVAL;
    int rc = check_ptr_array(*plan, (const void *const *)dev_part, has_part);
    if (rc != CCDC_OK) return rc;
    for (int k = 0; k < plan->K; ++k)
        if (has_part(*plan, k) && !host_part[k]) return CCDC_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    for (int k = 0; k < plan->K; ++k) {
        const size_t bytes = ccdc_partition_bytes(plan, k);
        if (!bytes) continue;
        cudaError_t e = cudaMemcpyAsync(dev_part[k], host_part[k], bytes, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    rc = ccdc_shuffle(plan, (const void *const *)dev_part, dev_coded, dev_out, dev_workspace, stream);
    if (rc != CCDC_OK) return rc;
    cudaError_t e = cudaMemcpyAsync(host_out, dev_out, ccdc_out_bytes(plan), cudaMemcpyDeviceToHost, st);
    return e == cudaSuccess ? CCDC_OK : cuda_fail(e);
}

}  // extern "C"

// ------------------------------------------------------------------------
// Allocation-free variant of ccdc_decode_reduce.
//
// Some callers cannot allocate device memory at the point where they shuffle:
// code that runs inside a region where cudaMalloc is forbidden or would
// synchronise the device (a latency-critical loop, a callback, a host thread
// that must not touch the allocator), or a host program whose memory budget
// was handed out in full at start-up.  For them the scratch of the split batch
// loop lives in the library image itself: a fixed array in device global
// memory that every GPU loading the library holds until the process exits.
//
// In host code the array's name is only a handle for the runtime, not a device
// address, so the address is looked up with cudaGetSymbolAddress, once per
// device with that device current, and that pointer is what the kernels get.
constexpr size_t CCDC_STATIC_SCRATCH_BYTES = 16u << 20;     // 16 MiB
static __device__ __align__(256) unsigned int g_static_scratch[CCDC_STATIC_SCRATCH_BYTES / 4];

namespace {
constexpr int MAX_DEVICES = 64;
std::atomic<void *> g_static_scratch_ptr[MAX_DEVICES];

// device address of the scratch array on the current device (set-up on first use)
int static_scratch_address(void **out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= MAX_DEVICES) return CCDC_ESIZE;
    void *p = g_static_scratch_ptr[dev].load(std::memory_order_acquire);
    if (!p) {
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return cuda_fail(e);
        g_static_scratch_ptr[dev].store(p, std::memory_order_release);
    }
    *out = p;
    return CCDC_OK;
}
}  // namespace

extern "C" {

size_t ccdc_static_scratch_bytes(void) { return CCDC_STATIC_SCRATCH_BYTES; }

int ccdc_decode_reduce_static(ccdc_plan_t *plan, const void *const *part, const void *coded, void *out,
                              void *stream) {
    if (!plan) return CCDC_EINVAL;
    if (ccdc_workspace_bytes(plan) > CCDC_STATIC_SCRATCH_BYTES) return CCDC_ESIZE;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (plan->device != dev) return CCDC_ESTATE;     // tables not uploaded here: uploading would allocate
    void *scratch = nullptr;
    int rc = static_scratch_address(&scratch);
    if (rc != CCDC_OK) return rc;
    return ccdc_decode_reduce(plan, part, coded, out, scratch, stream);
}

}  // extern "C"
