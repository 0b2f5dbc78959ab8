// The fused encode and the fused decode + reduce as persistent bulk-copy
// pipelines (sm_100a: cp.async.bulk global -> shared, completion on mbarriers).
//
// The register kernels of ccdc_kernels.cu keep every byte in flight in a
// register, and every thread block pays a memory latency for its table entries
// before its first load and another for its loads before its first result.
// With short segments (a few KiB per operand row) and few rows per block those
// latencies are most of a block's life.  Here the grid is three blocks per SM
// that stay: each block walks a contiguous range of output tiles ("items": a
// tile of a coded row for the encode; a tile of an output segment and one chunk
// of the job's batches for the decode).  The source rows of all its items form
// ONE sequence.  Two producer warps, each owning half of a ring of
// shared-memory stages (one lane per stage, the lanes in lockstep), stream that
// sequence in with bulk asynchronous copies, running ahead across item
// boundaries, so tens of KiB are in flight per block all the time and none of
// them in registers; 128 consumer threads fold the rows, in the order the
// scheme fixes, into three registers per word:
//     S  running sum over the files of the current operand   (pre-combining)
//     X  XOR over the operands of the current batch           (coding / decoding)
//     A  sum over the batches                                  (Eq. (1))
// and store X (encode) or A (decode) when an item's last row has been folded.
// The order of every addition is that of the register kernels and of the
// stepwise path (files ascending from the first file's value, batches
// ascending), so the results have the same bits.
//
// What to copy is a flat list the planner writes (ccdc_stream_row: source
// offset, valid length, role flags), one entry per source row of an output
// segment, so the producer does no table walking.
//
// A bulk copy needs 16-byte aligned addresses and sizes.  Segment starts are
// only 8-byte aligned when 4 does not divide s; such a row is copied from the
// 16-byte boundary below it and the consumers read it at an offset of two words.
// The bytes copied beyond a row's end stay inside the same file row (4 | len is
// required for this kernel family).
//
// Every wait is a bounded mbarrier poll.  A wait that runs out sets the plan's
// status word (ccdc_shuffle_status) and ends the block after its copies in
// flight have landed.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <utility>

#include "ccdc_internal.h"
#include "ccdc_stream.h"

namespace {

constexpr int CONSUMERS = 128;                  // threads that fold rows
constexpr int PRODUCERS = 2;                    // producer warps; each owns a contiguous share of the ring's stages
constexpr int ST_THREADS = CONSUMERS + 32 * PRODUCERS;
constexpr int TILE_WORDS = CCDC_STREAM_TILE_WORDS;      // words of a segment per item
constexpr int VECS = TILE_WORDS / (4 * CONSUMERS);      // 128-bit vectors (4 consecutive words) per consumer thread
constexpr int MAX_STAGES = 32;
constexpr int WAIT_LIMIT = 1 << 14;             // polls of an mbarrier before giving up (each may sleep up to SLEEP_NS)
constexpr unsigned SLEEP_NS = 200000;           // time a poll may suspend the thread waiting for the phase to complete
static_assert(TILE_WORDS % (4 * CONSUMERS) == 0, "tile must be a whole number of vectors per thread");

__device__ __forceinline__ unsigned smem_u32(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t *bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t *bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(SLEEP_NS)
        : "memory");
    return ok != 0;
}
// bounded wait; also gives up once another thread of the block has
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, unsigned parity, volatile int *abort_flag) {
    for (int i = 0; i < WAIT_LIMIT; ++i) {
        if (mbar_try(bar, parity)) return true;
        if ((i & 15) == 15 && *abort_flag) return false;
    }
    return false;
}
// bounded wait that does not look at the abort flag: used once, to let a copy in flight land
__device__ __forceinline__ bool mbar_wait_plain(uint64_t *bar, unsigned parity) {
    for (int i = 0; i < WAIT_LIMIT; ++i)
        if (mbar_try(bar, parity)) return true;
    return false;
}
// global -> shared bulk copy; `bytes` land on the barrier's transaction count
__device__ __forceinline__ void bulk_copy(void *dst_smem, const void *src, unsigned bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst_smem)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <bool F32>
__device__ __forceinline__ uint32_t add_word(uint32_t a, uint32_t b) {
    if (F32) return __float_as_uint(__fadd_rn(__uint_as_float(a), __uint_as_float(b)));
    return a + b;
}

// header of a stage, written by the producer before it arms the stage's barrier
constexpr unsigned H_END_ITEM = 1u << 24, H_SHIFT = 1u << 25;       // plus the row's CCDC_SROW_* flags << 16; low 16 bits: valid words
struct StageHeader {
    unsigned desc;
    int out_valid;          // END_ITEM rows: words of the item's output tile
    long long dst;          // END_ITEM rows: word offset of the item's output tile
};

struct StreamParams {
    const uint32_t *part[CCDC_MAX_K];
    const uint32_t *coded;          // source of the rows flagged CCDC_SROW_FROM_CODED
    uint32_t *out;                  // decode: [out rows][len] (the workspace when the batch loop is split); encode: coded buffer
    const ccdc_stream_cell *cells;
    const ccdc_stream_row *rows;
    const int *chunk_row0;          // [cells][nchunk + 1]
    const int *out_rows;            // decode on a node-sharded plan: the out rows to compute, else NULL
    int *status;
    long long nitems;
    long long tiles_per_seg;
    long long chunk_stride;         // decode with a split batch loop: words between two chunks' partial sums
    int r, nchunk, decode;
    int nstage, stage_bytes;
};

struct Shared {
    uint64_t full[MAX_STAGES];
    uint64_t empty[MAX_STAGES];
    StageHeader head[MAX_STAGES];
    unsigned long long total_rows;
    int abort_flag;
};

// cell, chunk and tile of an item
struct Item {
    long long cell, tile;
    int chunk;
};
__device__ __forceinline__ Item item_of(const StreamParams &p, long long it) {
    Item I;
    I.tile = it % p.tiles_per_seg; it /= p.tiles_per_seg;
    if (p.decode) {
        const int i = (int)(it % p.r); it /= p.r;
        I.chunk = (int)(it % p.nchunk);
        const long long li = it / p.nchunk;
        const long long orow = p.out_rows ? p.out_rows[li] : li;
        I.cell = orow * p.r + i;
    } else {
        I.chunk = 0;
        I.cell = it;
    }
    return I;
}
// rows of an item (0 if its tile lies beyond the segment's end)
__device__ __forceinline__ int item_rows(const StreamParams &p, const Item &I) {
    if (I.tile * TILE_WORDS >= p.cells[I.cell].seglen) return 0;
    const int *c = p.chunk_row0 + I.cell * (p.nchunk + 1) + I.chunk;
    return c[1] - c[0];
}

template <bool F32>
__global__ void __launch_bounds__(ST_THREADS)
k_stream(const __grid_constant__ StreamParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    Shared *sh = reinterpret_cast<Shared *>(smem);
    unsigned char *ring = smem + ((sizeof(Shared) + 127) & ~(size_t)127);
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;

    // this block's items
    const long long it0 = p.nitems * blockIdx.x / gridDim.x, it1 = p.nitems * (blockIdx.x + 1) / gridDim.x;
    pdl_trigger();
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.nstage; ++s) {
            mbar_init(&sh->full[s], 1);
            mbar_init(&sh->empty[s], CONSUMERS / 32);
        }
        sh->abort_flag = 0;
        sh->total_rows = 0ull;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    {   // rows of the block's sequence (plan tables only: nothing a kernel writes is read before pdl_wait)
        unsigned long long mine = 0;
        for (long long it = it0 + threadIdx.x; it < it1; it += ST_THREADS) mine += (unsigned long long)item_rows(p, item_of(p, it));
        for (int o = 16; o > 0; o >>= 1) mine += __shfl_down_sync(0xffffffffu, mine, o);
        if (lane == 0 && mine) atomicAdd(&sh->total_rows, mine);
    }
    __syncthreads();
    const long long total = (long long)sh->total_rows;
    pdl_wait();
    volatile int *abort_flag = &sh->abort_flag;

    if (warp >= CONSUMERS / 32) {
        // ---------------- producers: warp w owns stages [w*G, (w+1)*G), G = nstage / PRODUCERS, lane l of it stage
        // w*G + l.  Its lanes work in lockstep on one row each (round k: rows k*nstage + stage), so a round
        // costs one pass of the instruction stream for G rows; the warp refills its stages when all of them
        // have been released, while the consumers are busy with the other warp's stages.
        const int pw = warp - CONSUMERS / 32;
        const int G = p.nstage / PRODUCERS;
        if (lane < G) {
            const unsigned mask = G >= 32 ? 0xffffffffu : ((1u << G) - 1u);
            const int st = pw * G + lane;
            long long it = it0 - 1, first = 0;      // current item and the sequence index of its first row
            int nrows = 0;                          // rows of the current item
            Item I = {0, 0, 0};
            ccdc_stream_cell C = {0, 0, 0, 0};
            long long row_base = 0;
            bool ok = true;
            unsigned round = 0;
            for (long long n0 = (long long)pw * G; n0 < total && ok; n0 += p.nstage, ++round) {     // n0: the warp's first row of the round
                const long long n = n0 + lane;
                const bool mine = n < total;
                ccdc_stream_row R = {0, 0, 0};
                long long tile0 = 0;
                int x = 0;
                if (mine) {
                    while (n >= first + nrows) {    // on to the item that holds row n (items without rows are skipped)
                        first += nrows;
                        ++it;
                        I = item_of(p, it);
                        nrows = item_rows(p, I);
                        if (nrows) {
                            C = p.cells[I.cell];
                            row_base = C.row0 + p.chunk_row0[I.cell * (p.nchunk + 1) + I.chunk];
                        }
                    }
                    x = (int)(n - first);
                    R = p.rows[row_base + x];
                    tile0 = I.tile * TILE_WORDS;
                }
                const int valid = mine ? (int)max(0LL, min((long long)TILE_WORDS, (long long)R.vl - tile0)) : 0;
                const uint32_t *src = ((R.flags & CCDC_SROW_FROM_CODED) ? p.coded : p.part[C.src_node]) + R.off + tile0;
                const uintptr_t g = reinterpret_cast<uintptr_t>(src);
                const unsigned shift = valid > 0 ? (unsigned)(g & 15u) : 0u;
                if (round > 0) {                    // all of the warp's stages released by the consumers?
                    bool all = false;
                    for (int i = 0; i < WAIT_LIMIT && !all; ++i) {
                        const bool freed = !mine || mbar_try(&sh->empty[st], (round - 1) & 1u);
                        all = __all_sync(mask, freed);
                        if (!all && (i & 15) == 15 && *abort_flag) break;
                    }
                    ok = all;
                }
                if (!ok || !mine) continue;         // (ok is the same in every lane: the loop ends for all of them)
                unsigned desc = (unsigned)valid | ((unsigned)R.flags << 16) | (shift ? H_SHIFT : 0u);
                if (x == nrows - 1) {
                    desc |= H_END_ITEM;
                    sh->head[st].dst = C.dst_off + tile0 + (long long)I.chunk * p.chunk_stride;
                    sh->head[st].out_valid = (int)min((long long)TILE_WORDS, (long long)C.seglen - tile0);
                }
                sh->head[st].desc = desc;
                if (valid <= 0) {
                    mbar_expect_tx(&sh->full[st], 0);               // nothing to copy: the phase completes at once
                } else {
                    const unsigned bytes = (shift + (unsigned)valid * 4u + 15u) & ~15u;
                    mbar_expect_tx(&sh->full[st], bytes);
                    bulk_copy(ring + (size_t)st * p.stage_bytes, reinterpret_cast<const void *>(g - shift), bytes, &sh->full[st]);
                }
            }
            if (!ok) {
                if (lane == 0) { *abort_flag = 1; atomicExch(p.status, 1); }
                // let the copy this lane may have in flight (filled in the round before the one that gave up) land
                // before the block's shared memory is given up
                if (round >= 2) mbar_wait_plain(&sh->full[st], (round - 2) & 1u);
            }
        }
        return;
    }

    // ---------------- consumers: thread t owns words 4t .. 4t+3 of every 512-word slice of the tile
    uint32_t S[VECS][4], X[VECS][4], A[VECS][4];
#pragma unroll
    for (int v = 0; v < VECS; ++v)
#pragma unroll
        for (int c = 0; c < 4; ++c) S[v][c] = X[v][c] = A[v][c] = 0u;
    int st = 0;
    unsigned phase = 0;
    for (long long n = 0; n < total; ++n, st = st + 1 == p.nstage ? 0 : st + 1, phase ^= st == 0 ? 1u : 0u) {
        if (!mbar_wait(&sh->full[st], phase, abort_flag)) {
            if (!*abort_flag) { *abort_flag = 1; atomicExch(p.status, 1); }
            return;
        }
        const unsigned d = sh->head[st].desc;
        const int valid = (int)(d & 0xffffu);
        const unsigned f = (d >> 16) & 0xffu;
        const bool shifted = (d & H_SHIFT) != 0;        // the row starts 8 bytes into the stage: two 64-bit loads per vector
        const uint32_t *words = reinterpret_cast<const uint32_t *>(ring + (size_t)st * p.stage_bytes + (shifted ? 8 : 0));
        uint32_t in[VECS][4];
#pragma unroll
        for (int v = 0; v < VECS; ++v) {
            const int w = (v * CONSUMERS + (int)threadIdx.x) * 4;
            const int left = valid - w;                 // even: 4 or more, 2, or none
            in[v][0] = in[v][1] = in[v][2] = in[v][3] = 0u;
            if (left >= 4 && !shifted) {
                const uint4 q = *reinterpret_cast<const uint4 *>(words + w);
                in[v][0] = q.x; in[v][1] = q.y; in[v][2] = q.z; in[v][3] = q.w;
            } else if (left >= 2) {
                const uint2 q = *reinterpret_cast<const uint2 *>(words + w);
                in[v][0] = q.x; in[v][1] = q.y;
                if (left >= 4) {
                    const uint2 q2 = *reinterpret_cast<const uint2 *>(words + w + 2);
                    in[v][2] = q2.x; in[v][3] = q2.y;
                }
            }
        }
        const bool end = (d & H_END_ITEM) != 0;
        const long long dst_off = end ? sh->head[st].dst : 0;
        const int out_valid = end ? sh->head[st].out_valid : 0;
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh->empty[st]);     // the stage is free again: everything needed is in registers
        // the row's role is the same for every word: branch once, not per vector
        if (f & CCDC_SROW_CODED) {
#pragma unroll
            for (int v = 0; v < VECS; ++v)
#pragma unroll
                for (int c = 0; c < 4; ++c) X[v][c] = in[v][c];
        } else {
            if (f & CCDC_SROW_FIRST_FILE) {
#pragma unroll
                for (int v = 0; v < VECS; ++v)
#pragma unroll
                    for (int c = 0; c < 4; ++c) S[v][c] = in[v][c];
            } else {
#pragma unroll
                for (int v = 0; v < VECS; ++v)
#pragma unroll
                    for (int c = 0; c < 4; ++c) S[v][c] = add_word<F32>(S[v][c], in[v][c]);
            }
            if (f & CCDC_SROW_LAST_FILE) {
                if (f & CCDC_SROW_FIRST_OP) {
#pragma unroll
                    for (int v = 0; v < VECS; ++v)
#pragma unroll
                        for (int c = 0; c < 4; ++c) X[v][c] = S[v][c];
                } else {
#pragma unroll
                    for (int v = 0; v < VECS; ++v)
#pragma unroll
                        for (int c = 0; c < 4; ++c) X[v][c] ^= S[v][c];
                }
            }
        }
        if ((f & (CCDC_SROW_LAST_FILE | CCDC_SROW_LAST_OP)) == (CCDC_SROW_LAST_FILE | CCDC_SROW_LAST_OP)) {
#pragma unroll
            for (int v = 0; v < VECS; ++v)
#pragma unroll
                for (int c = 0; c < 4; ++c) A[v][c] = add_word<F32>(A[v][c], X[v][c]);
        }
        if (end) {
            // The item's tile is complete.  Encode: the coded words are X itself (adding the one batch to zero
            // would turn -0.0 into +0.0).  Decode: the sum over the batches.  The output tile may itself start
            // 8 bytes off a 16-byte boundary (segments of 4k+2 words): 64-bit stores then.
            uint32_t *dst = p.out + dst_off;
            const bool dst16 = (reinterpret_cast<uintptr_t>(dst) & 15u) == 0;
#pragma unroll
            for (int v = 0; v < VECS; ++v) {
                const int w = (v * CONSUMERS + (int)threadIdx.x) * 4;
                const int left = out_valid - w;
                uint32_t o[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) { o[c] = p.decode ? A[v][c] : X[v][c]; A[v][c] = 0u; }
                if (left >= 4 && dst16) {
                    *reinterpret_cast<uint4 *>(dst + w) = make_uint4(o[0], o[1], o[2], o[3]);
                } else if (left >= 2) {
                    *reinterpret_cast<uint2 *>(dst + w) = make_uint2(o[0], o[1]);
                    if (left >= 4) *reinterpret_cast<uint2 *>(dst + w + 2) = make_uint2(o[2], o[3]);
                }
            }
        }
    }
}

template <typename... KArgs, typename... Args>
cudaError_t launch_kernel(void (*kernel)(KArgs...), long long grid, int block, size_t smem, cudaStream_t st, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// stage size and count for a plan: a stage holds one tile of a row plus the alignment slack
void ring_shape(const ccdc_plan_s &P, int *nstage, int *stage_bytes, size_t *smem) {
    const long long tile = std::min<long long>(TILE_WORDS, (P.s + 1) / 2 * 2);
    *stage_bytes = (int)((tile * 4 + 16 + 127) / 128 * 128);
    const size_t fixed = (sizeof(Shared) + 127) / 128 * 128;
    const long long n = (long long)(((size_t)CCDC_STREAM_SMEM_BYTES - fixed) / *stage_bytes);
    *nstage = (int)std::max<long long>(PRODUCERS, std::min<long long>(n, MAX_STAGES) / PRODUCERS * PRODUCERS);
    *smem = fixed + (size_t)*nstage * *stage_bytes;
}

int launch_stream(const ccdc_plan_s &P, StreamParams &sp, cudaStream_t st) {
    size_t smem = 0;
    ring_shape(P, &sp.nstage, &sp.stage_bytes, &smem);
    if (sp.nitems <= 0) return CCDC_OK;
    const long long blocks = std::min<long long>(sp.nitems, (long long)P.sm_count * 3);
    const bool f32 = P.dtype == CCDC_F32;
    cudaError_t e = f32 ? cudaFuncSetAttribute(k_stream<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                        : cudaFuncSetAttribute(k_stream<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return ccdc_internal_cuda_fail((int)e);
    if (f32) launch_kernel(k_stream<true>, blocks, ST_THREADS, smem, st, sp);
    else launch_kernel(k_stream<false>, blocks, ST_THREADS, smem, st, sp);
    ccdc_internal_count_launch();
    e = cudaGetLastError();
    return e == cudaSuccess ? CCDC_OK : ccdc_internal_cuda_fail((int)e);
}

void fill_common(const ccdc_plan_s &P, const void *const *part, const ccdc_stream_table &T, StreamParams &sp) {
    std::memset(&sp, 0, sizeof(sp));
    for (int k = 0; k < P.K; ++k) sp.part[k] = static_cast<const uint32_t *>(part[k]);
    sp.status = P.d_status;
    sp.cells = T.d_cells; sp.rows = T.d_rows; sp.chunk_row0 = T.d_chunk_row0;
    sp.tiles_per_seg = (P.s + TILE_WORDS - 1) / TILE_WORDS;
    sp.r = P.r;
}

}  // namespace

long long ccdc_stream_tile_words() { return TILE_WORDS; }

bool ccdc_stream_supported(const ccdc_plan_s &P) {
    if (P.compression_mode || P.device_has_bulk_copies == 0) return false;
    if (P.len % 4 != 0 || P.s % 2 != 0) return false;               // rows 16-byte aligned, segments 8-byte aligned
    if (P.s > (1LL << 30)) return false;                            // valid lengths are ints
    // the flat row lists (16 bytes per source row of every output segment and coded row) must stay modest
    const long long dec_rows = P.J * P.K * P.r * P.nterm * (1 + (long long)(P.r - 1) * P.b);
    const long long enc_rows = P.nround * (P.r + 1) * P.r * P.b;
    return (dec_rows + enc_rows) * (long long)sizeof(ccdc_stream_row) <= (1LL << 30);
}

int ccdc_stream_decode(const ccdc_plan_s &P, const void *const *part, const void *coded, void *out, void *ws,
                       cudaStream_t st) {
    StreamParams sp;
    fill_common(P, part, P.dec_stream, sp);
    sp.coded = static_cast<const uint32_t *>(coded);
    sp.decode = 1;
    sp.nchunk = P.nchunk;
    sp.out = static_cast<uint32_t *>(P.nchunk == 1 ? out : ws);
    sp.chunk_stride = P.nchunk == 1 ? 0 : P.J * P.K * P.len;
    sp.out_rows = P.shard_world > 1 ? P.d_out_rows : nullptr;
    const long long nlist = P.shard_world > 1 ? (long long)P.out_rows.size() : P.J * P.K;
    sp.nitems = nlist * P.nchunk * P.r * sp.tiles_per_seg;
    return launch_stream(P, sp, st);
}

int ccdc_stream_encode(const ccdc_plan_s &P, const void *const *part, void *coded, cudaStream_t st) {
    StreamParams sp;
    fill_common(P, part, P.enc_stream, sp);
    sp.decode = 0;
    sp.nchunk = 1;
    sp.out = static_cast<uint32_t *>(coded);
    sp.nitems = (long long)P.enc_stream.cells.size() * sp.tiles_per_seg;
    return launch_stream(P, sp, st);
}
