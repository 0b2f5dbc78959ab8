// Map phase of the linear-regression workload (Section III, "Map phase"), the
// version that reads X exactly once:  g_n = X_n^T (X_n w - y_n).
//
// A thread-block cluster of C = d / 2048 blocks owns a file; block c owns the
// columns [2048 c, 2048 (c+1)).  X arrives by TMA in row blocks of 8 rows: a
// stage is the block's 8 x 2048 slab (32 KiB, one 3-D box), six stages ring
// through shared memory; a fetch warp refills a stage right after the block
// barrier that follows its last use.  For every row block:
//   1. first product: each warp multiplies its 256 columns of the slab by w on
//      the tensor cores (mma.sync m16n8k16, A by ldmatrix, w held in registers
//      as B fragments) and leaves 8 partial dot products in shared memory;
//   2. a send warp adds the 8 warps' partials (a fixed tree) and hands the
//      block's 8 partial dots to all blocks of the cluster through
//      distributed shared memory (asynchronous remote stores
//      that count their bytes on the receiver's mbarrier); a receive warp adds
//      the C blocks' partials in a fixed order, subtracts y, and splits the
//      residual u into three bf16 terms (u = hi + mid + lo);
//   3. second product: each warp multiplies the transposed slab (A by
//      ldmatrix.trans, mma.sync m16n8k8) by the three terms (columns 0..2 of B)
//      and accumulates its 256 gradient columns in registers.
// The loop is software pipelined behind one block barrier per row block: the
// first product runs two row blocks ahead of the second, a row block's partial
// dots are sent in the iteration that computes them and received in the next.
// The slab is read from shared memory twice and from HBM once.
//
// Summation order.  A file is cut into UF units of rows/UF rows (UF = 4 when
// rows is a multiple of 32, else 1).  Within a unit the row blocks accumulate
// in order; the file's gradient is ((unit0 + unit1) + unit2) + unit3.  Units
// are the grain of the work split over the clusters (contiguous, equal
// shares), so that the clusters finish together; because the order above does
// not depend on where a share ends, every replica of a file gets the same bits
// whichever node maps it.  A file that straddles two shares has its pieces
// written to a workspace and added, in the same order, by k_map_combine.
//
// Every wait is bounded (mbarrier polls with a limit); a wait that runs out
// sets the status word, and the thread runs to the kernel's end on stale data
// with all its later waits cut to a few polls.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>

#include "ccdc_internal.h"
#include "ccdc_map_cluster.h"

namespace {

constexpr int WARPS = 8;                            // compute warps
constexpr int THREADS = WARPS * 32 + 96;            // + the send, receive and fetch warps
constexpr int RB = 8;                               // rows per row block
constexpr int COLS_CTA = 2048;                      // columns per block
constexpr int COLS_WARP = COLS_CTA / WARPS;         // 256
constexpr int KSTEPS = COLS_WARP / 32;              // 8 MMAs per warp in the first product (32 columns each)
constexpr int NBLK = COLS_WARP / 8;                 // 32 MMAs per warp in the second (8 columns each)
constexpr int CHUNKS_CTA = COLS_CTA / 64;           // 32 chunks of 64 columns (128 bytes)
constexpr int STAGE_BYTES = CHUNKS_CTA * RB * 128;  // 32 KiB
constexpr int STAGES = 6;
constexpr int XBUF = 4;                             // exchange buffers: a peer may run up to 3 row blocks ahead
constexpr int MAX_CLUSTER = 8;
constexpr int MAX_SPLIT = 160;                      // listed files cut between two shares (at most one per share)
constexpr int WAIT_LIMIT = 1 << 20;

struct ClusterParams {
    CUtensorMap tmap[CCDC_MAX_K];       // node k: X as (64 columns, files * rows, d / 64 chunks)
    const float *y[CCDC_MAX_K];         // node k: [local file][rows]
    float *part[CCDC_MAX_K];            // node k: [local file][d]
    long long first_job[CCDC_MAX_K + 1];// jobs are (node, local file), node-major
    const uint16_t *w;                  // [d] bf16
    float *pieces;                      // [jobs][UF][d]: pieces of files that straddle two shares
    int *status;
    long long njobs, rows, d;
    int K, UF, nclusters;
    int nsplit;                         // files cut between shares, listed below; -1: not listed, look at every file
    int split_jobs[MAX_SPLIT];
};

__device__ __forceinline__ unsigned smem_u32(const void *ptr) { return (unsigned)__cvta_generic_to_shared(ptr); }

__device__ __forceinline__ int node_of_job(const ClusterParams &p, long long job) {
    int k = 0;
    while (k + 1 < p.K && job >= p.first_job[k + 1]) ++k;
    return k;
}

// first unit of cluster c's share: equal contiguous shares of the njobs * UF units
__host__ __device__ __forceinline__ long long share_start(long long units, int nclusters, int c) {
    return units * c / nclusters;
}
// the cluster whose share holds unit x
__host__ __device__ __forceinline__ int share_of_unit(long long units, int nclusters, long long x) {
    int c = (int)(x * nclusters / units);
    while (c + 1 < nclusters && share_start(units, nclusters, c + 1) <= x) ++c;
    while (c > 0 && share_start(units, nclusters, c) > x) --c;
    return c;
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// bounded wait for the bytes a barrier expects: the block's own TMA copies, or the peers' asynchronous stores
// (both are made visible to the waiter by the barrier's completion)
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, unsigned parity, int limit) {
    const unsigned addr = smem_u32(bar);
    for (int i = 0; i < limit; ++i) {
        unsigned ok;
        asm volatile(
            "{\n"
            ".reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
            "selp.u32 %0, 1, 0, p;\n"
            "}\n"
            : "=r"(ok)
            : "r"(addr), "r"(parity)
            : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ unsigned peer_addr(unsigned local, unsigned rank) {
    unsigned remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    return remote;
}
// asynchronous store of one word into a peer's shared memory; on landing it counts 4 bytes on the peer's barrier
__device__ __forceinline__ void peer_store(unsigned remote, float v, unsigned remote_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
                 ::"r"(remote), "r"(__float_as_uint(v)), "r"(remote_bar) : "memory");
}
// block barrier of the compute, receive and fetch warps (the send warp does not take part)
__device__ __forceinline__ void block_sync() {
    asm volatile("bar.sync 1, %0;" ::"n"(THREADS - 32) : "memory");
}
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ unsigned cluster_rank() {
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void tma_slab(unsigned dst, const CUtensorMap *map, int row, int chunk, uint64_t *bar,
                                         uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3, %4}], [%5], %6;"
        ::"r"(dst), "l"(map), "r"(0), "r"(row), "r"(chunk), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(unsigned addr, uint32_t (&v)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(unsigned addr, uint32_t (&v)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_k16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_k8(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(b0));
}

// walks the row blocks of a share in order: file (node k, local index `file`), unit ui, row block rb
struct Cursor {
    long long job, file, rb;
    int ui, k;
    __device__ void start(const ClusterParams &p, long long unit) {
        job = unit / p.UF;
        ui = (int)(unit - job * p.UF);
        rb = 0;
        k = node_of_job(p, job);
        file = job - p.first_job[k];
    }
    __device__ void next(const ClusterParams &p, long long rbu) {
        if (++rb < rbu) return;
        rb = 0;
        if (++ui < p.UF) return;
        ui = 0;
        ++job;
        ++file;
        while (k + 1 < p.K && job >= p.first_job[k + 1]) { ++k; file = job - p.first_job[k]; }
    }
    __device__ long long row(long long rbu) const { return (ui * rbu + rb) * RB; }     // first row inside the file
};

__global__ void __launch_bounds__(THREADS, 1)
k_map_cluster(const __grid_constant__ ClusterParams p) {
    extern __shared__ unsigned char sh_raw[];
    __shared__ __align__(8) uint64_t full[STAGES];      // the stage's slab has landed
    __shared__ __align__(8) uint64_t xbar[XBUF];        // all blocks' partial dots of a row block have landed
    __shared__ __align__(8) uint64_t pbar[4];           // the 8 warps' partial dots of a row block are in sh_part
    __shared__ float sh_part[4][WARPS][RB];
    __shared__ float xch[XBUF][MAX_CLUSTER][RB];
    __shared__ uint32_t sh_u[2][3][RB / 2];             // hi / mid / lo terms of u as bf16 pairs, two row blocks
    __shared__ __align__(16) float sh_tot[COLS_CTA];    // sum of the file's units so far

    const unsigned ring = (smem_u32(sh_raw) + 1023u) & ~1023u;   // the 128-byte swizzle wants 1 KiB alignment
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int C = (int)(p.d / COLS_CTA);
    const unsigned rank = cluster_rank();
    const int cid = blockIdx.x / C;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init(&full[s], 1);
        for (int s = 0; s < XBUF; ++s) mbar_init(&xbar[s], 1);
        for (int s = 0; s < 4; ++s) mbar_init(&pbar[s], WARPS);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    cluster_sync();         // no block signals a peer's barrier before it exists

    const long long units = p.njobs * p.UF;
    const long long u0 = share_start(units, p.nclusters, cid), u1 = share_start(units, p.nclusters, cid + 1);
    const long long rbu = p.rows / p.UF / RB;           // row blocks per unit
    const long long nrb = (u1 - u0) * rbu;              // row blocks of this cluster's share
    bool timed_out = false;

    if (warp == WARPS + 2) {
        // ================= the fetch warp: one lane keeps the ring full, one 32 KiB box per row block ==========
        uint64_t policy;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
        Cursor load;            // the next row block to fetch
        load.start(p, u0);
        long long nload = 0;
        int slot0 = 0;
        auto fetch = [&]() {
            mbar_expect_tx(&full[slot0], STAGE_BYTES);
            tma_slab(ring + slot0 * STAGE_BYTES, &p.tmap[load.k], (int)(load.file * p.rows + load.row(rbu)),
                     (int)(rank * CHUNKS_CTA), &full[slot0], policy);
            load.next(p, rbu);
            ++nload;
            if (++slot0 == STAGES) slot0 = 0;
        };
        if (lane == 0)
            while (nload < STAGES && nload < nrb) fetch();
        block_sync();
        for (long long i = 0; i < nrb; ++i) {
            block_sync();    // the second product of row block i-1 is over: its stage can be refilled
            if (lane == 0 && i > 0 && nload < nrb) fetch();
            __syncwarp();
        }
    } else if (warp == WARPS) {
        // ================= the send warp =================
        // lane l = (row r = l % 8, quarter q = l / 8)
        // send: add the 8 warps' partial dots of row block j (a fixed tree) and store the sum into the exchange
        // buffer of every block of the cluster, this lane serving blocks q and q + 4
        const int xr = lane & 7, xq = lane >> 3;
        const unsigned peer_lo = peer_addr(smem_u32(&xch[0][0][0]), xq < C ? xq : 0);
        const unsigned peer_hi = peer_addr(smem_u32(&xch[0][0][0]), xq + 4 < C ? xq + 4 : 0);
        const unsigned bar_off = smem_u32(&xbar[0]) - smem_u32(&xch[0][0][0]);    // same offset in every block
        auto send = [&](long long j) {
            const int b = (int)(j & 3), xs = (int)(j & (XBUF - 1));
            if (!mbar_wait(&pbar[b], (unsigned)((j >> 2) & 1), timed_out ? 64 : WAIT_LIMIT)) timed_out = true;
            float s = sh_part[b][xq][xr] + sh_part[b][xq + 4][xr];
            s += __shfl_xor_sync(0xffffffffu, s, 8);
            s += __shfl_xor_sync(0xffffffffu, s, 16);
            if (lane == 0) mbar_expect_tx(&xbar[xs], 4u * RB * C);      // 8 words from every block
            const unsigned word = (unsigned)(((xs * MAX_CLUSTER + (int)rank) * RB + xr) * 4);
            const unsigned bar = bar_off + (unsigned)(xs * 8);
            if (xq < C) peer_store(peer_lo + word, s, peer_lo + bar);
            if (xq + 4 < C) peer_store(peer_hi + word, s, peer_hi + bar);
        };
        // The send warp runs free of the block barrier: it follows the compute warps through pbar alone.  (A row
        // block's buffer in sh_part is rewritten four row blocks later, which the compute warps reach only after
        // the receive of a later row block, i.e. after this warp's later sends.)
        for (long long j = 0; j < nrb; ++j) send(j);
    } else if (warp == WARPS + 1) {
        // ================= the receive warp =================
        const int xr = lane & 7, xq = lane >> 3;
        // receive: add the blocks' partial dots of row block j (a fixed tree), subtract y and leave the three bf16
        // terms of the residual in sh_u[j % 2]
        Cursor rcv;             // the next row block to receive
        rcv.start(p, u0);
        const float *ybase = p.y[rcv.k] + rcv.file * p.rows;
        float yv = 0.f;
        if (lane < RB && nrb > 0) yv = __ldg(ybase + rcv.row(rbu) + lane);
        auto receive = [&](long long j) {
            const int xs = (int)(j & (XBUF - 1));
            if (!mbar_wait(&xbar[xs], (unsigned)((j / XBUF) & 1), timed_out ? 64 : WAIT_LIMIT)) timed_out = true;
            float dot = xq < C ? xch[xs][xq][xr] : 0.f;
            if (xq + 4 < C) dot += xch[xs][xq + 4][xr];
            dot += __shfl_xor_sync(0xffffffffu, dot, 8);
            dot += __shfl_xor_sync(0xffffffffu, dot, 16);
            const long long file_was = rcv.job;
            rcv.next(p, rbu);
            if (rcv.job != file_was && j + 1 < nrb) ybase = p.y[rcv.k] + rcv.file * p.rows;
            if (lane < RB) {
                float rest = dot - yv;
                uint16_t term[3];
                for (int e = 0; e < 3; ++e) {
                    const __nv_bfloat16 h = __float2bfloat16_rn(rest);
                    term[e] = __bfloat16_as_ushort(h);
                    rest = rest - __bfloat162float(h);      // exact in fp32
                }
                for (int e = 0; e < 3; ++e) reinterpret_cast<uint16_t *>(sh_u[j & 1][e])[lane] = term[e];
                if (j + 1 < nrb) yv = __ldg(ybase + rcv.row(rbu) + lane);       // used an iteration later
            }
        };

        if (nrb > 0) receive(0);
        block_sync();
        for (long long i = 0; i < nrb; ++i) {
            block_sync();    // the second product of row block i-1 is over: sh_u[(i+1) % 2] is free
            if (i + 1 < nrb) receive(i + 1);
        }
    } else {
        // ================= the eight compute warps =================
        const int g = lane / 4, t = lane % 4;
        // w as B fragments of the first product.  An MMA covers 32 columns c .. c+31: tile rows 0..7 are the 8 rows
        // of the slab times columns c .. c+15 (w in column 0 of B), tile rows 8..15 the same rows times columns
        // c+16 .. c+31 (w in column 1 of B).  Lanes g = 0, 1 hold the two columns of B.
        uint32_t wf[KSTEPS][2];
        {
            const uint32_t *w32 = reinterpret_cast<const uint32_t *>(p.w) + (rank * COLS_CTA + warp * COLS_WARP) / 2;
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                wf[ks][0] = g < 2 ? __ldg(w32 + ks * 16 + g * 8 + t) : 0u;
                wf[ks][1] = g < 2 ? __ldg(w32 + ks * 16 + g * 8 + 4 + t) : 0u;
            }
        }
        // ldmatrix: lane l points at row l % 8 of a 16-byte unit of a chunk; in shared memory a 128-byte line is
        // (chunk, row) and its units are permuted by the row number (the TMA swizzle).
        // First product: matrices 0..3 of an x4 load are units j, j+2, j+1, j+3 (the A fragment order above).
        // Second product (transposed load): matrices 0..3 are units j .. j+3 = four blocks of 8 columns.
        const unsigned lrow = (unsigned)(lane & 7), lm = (unsigned)(lane >> 3);
        const unsigned lane_base = (unsigned)(warp * 4 * RB * 128) + lrow * 128;
        const unsigned unit1 = ((lm & 1) << 1) | (lm >> 1), unit2 = lm;

        // first product of the row block in `slot`; lanes t = 0 leave row g's partial dot product in dst[g]
        auto first_product = [&](int slot, float *dst, uint64_t *ready) {
            const unsigned stage = ring + slot * STAGE_BYTES + lane_base;
            float e0[4] = {0.f, 0.f, 0.f, 0.f}, e1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                uint32_t a[4];
                ldmatrix_x4(stage + (ks >> 1) * (RB * 128) + ((((ks & 1) * 4 + unit1) ^ lrow) << 4), a);
                if (ks & 1) mma_k16(e1, a, wf[ks][0], wf[ks][1]);
                else mma_k16(e0, a, wf[ks][0], wf[ks][1]);
            }
            if (t == 0) dst[g] = (e0[0] + e1[0]) + (e0[3] + e1[3]);     // D[g][0] + D[g+8][1]
            __syncwarp();
            if (lane == 0) mbar_arrive(ready);      // this warp's 8 partial dots are in place
        };
        // this unit's gradient: tile j of the second product is D[16 columns][n], n = 0, 1, 2 the three terms of u;
        // lane (g, t) holds columns 16 j + g (acc[j][0..1]) and 16 j + 8 + g (acc[j][2..3]) at n = 2t, 2t + 1
        float acc[NBLK / 2][4];
#pragma unroll
        for (int j = 0; j < NBLK / 2; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;

        // The pipeline: F = first product, S = send, R = receive, G = second product.  Iteration i runs F(i+2),
        // then S(i+2) as soon as all warps' partial dots are in (an mbarrier, no block barrier), R(i+1) and G(i),
        // behind ONE block barrier: three stages hold data, three are in flight.
        int slot1 = 0;          // stage of the next first product
        unsigned round1 = 0;
        long long nfirst = 0;
        auto first_next = [&]() {
            if (nfirst >= nrb) return;
            if (!mbar_wait(&full[slot1], round1 & 1u, timed_out ? 64 : WAIT_LIMIT)) timed_out = true;
            first_product(slot1, sh_part[nfirst & 3][warp], &pbar[nfirst & 3]);
            ++nfirst;
            if (++slot1 == STAGES) { slot1 = 0; ++round1; }
        };
        first_next();
        first_next();
        block_sync();

        Cursor cur;             // the row block of the second product
        cur.start(p, u0);
        int slot2 = 0;
        for (long long i = 0; i < nrb; ++i) {
            block_sync();    // u of row block i is in place; G(i-1) is over everywhere
            first_next();       // F(i+2)

            // ---- second product G(i): the transposed slab [256 columns x 8 rows] times (hi, mid, lo) [8 rows x 3]
            {
                const unsigned stage = ring + slot2 * STAGE_BYTES + lane_base;
                const uint32_t b0 = g < 3 ? sh_u[i & 1][g][t] : 0u;
#pragma unroll
                for (int q = 0; q < NBLK / 4; ++q) {
                    uint32_t a[4];
                    ldmatrix_x4_trans(stage + (q >> 1) * (RB * 128) + ((((q & 1) * 4 + unit2) ^ lrow) << 4), a);
                    mma_k8(acc[2 * q], a[0], a[1], b0);
                    mma_k8(acc[2 * q + 1], a[2], a[3], b0);
                }
                if (++slot2 == STAGES) slot2 = 0;
            }

            // ---- end of a unit: fold the three terms, then add the unit to the file's sum or set it aside
            if (cur.rb == rbu - 1) {
                const long long unit = u0 + i / rbu;
                const bool prefix = cur.job * p.UF >= u0;       // this share holds the file from its first unit on
                const bool last_here = cur.ui == p.UF - 1 || unit == u1 - 1;
                float *dst = nullptr;
                if (!prefix) dst = p.pieces + (cur.job * p.UF + cur.ui) * p.d;
                else if (last_here) dst = cur.ui == p.UF - 1 ? p.part[cur.k] + cur.file * p.d : p.pieces + cur.job * p.UF * p.d;
                float *tot = sh_tot + warp * COLS_WARP;         // this warp's columns; also stages the coalesced store
                const bool add = prefix && cur.ui != 0;
                float v[NBLK / 2][2];
#pragma unroll
                for (int j = 0; j < NBLK / 2; ++j) {
                    const float lo0 = __shfl_down_sync(0xffffffffu, acc[j][0], 1);   // n = 2 lives in lane t = 1
                    const float lo1 = __shfl_down_sync(0xffffffffu, acc[j][2], 1);
                    v[j][0] = (acc[j][0] + acc[j][1]) + lo0;
                    v[j][1] = (acc[j][2] + acc[j][3]) + lo1;
                    acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;
                }
                if (t == 0) {
                    if (add) {
                        float old[NBLK / 2][2];
#pragma unroll
                        for (int j = 0; j < NBLK / 2; ++j) { old[j][0] = tot[16 * j + g]; old[j][1] = tot[16 * j + 8 + g]; }
#pragma unroll
                        for (int j = 0; j < NBLK / 2; ++j) { v[j][0] = old[j][0] + v[j][0]; v[j][1] = old[j][1] + v[j][1]; }
                    }
#pragma unroll
                    for (int j = 0; j < NBLK / 2; ++j) { tot[16 * j + g] = v[j][0]; tot[16 * j + 8 + g] = v[j][1]; }
                }
                __syncwarp();
                if (dst) {
                    float4 *out4 = reinterpret_cast<float4 *>(dst + rank * COLS_CTA + warp * COLS_WARP);
                    const float4 *tot4 = reinterpret_cast<const float4 *>(tot);
                    out4[lane] = tot4[lane];
                    out4[lane + 32] = tot4[lane + 32];
                }
                __syncwarp();
            }
            cur.next(p, rbu);
        }
    }
    if (timed_out) atomicExch(p.status, 1);
    cluster_sync();             // no block leaves while a peer may still store into its shared memory
}

// Files whose units fell into two or more shares: out = ((piece 0 + unit b0) + unit b0+1) + ..., where
// piece 0 is the sum of units 0 .. b0-1 left by the share that held the file's first unit.
__global__ void k_map_combine(const __grid_constant__ ClusterParams p) {
    const long long job = p.nsplit >= 0 ? p.split_jobs[blockIdx.x] : blockIdx.x;
    const long long units = p.njobs * p.UF, first = job * p.UF;
    const int c0 = share_of_unit(units, p.nclusters, first);
    if (c0 == share_of_unit(units, p.nclusters, first + p.UF - 1)) return;     // mapped whole by one share
    const int b0 = (int)(share_start(units, p.nclusters, c0 + 1) - first);
    const int k = node_of_job(p, job);
    const long long file = job - p.first_job[k];
    const float4 *src = reinterpret_cast<const float4 *>(p.pieces + first * p.d);
    float4 *dst = reinterpret_cast<float4 *>(p.part[k] + file * p.d);
    const long long n4 = p.d / 4;
    for (long long j = blockIdx.y * (long long)blockDim.x + threadIdx.x; j < n4; j += (long long)gridDim.y * blockDim.x) {
        float4 s = src[j];
        for (int ui = b0; ui < p.UF; ++ui) {
            const float4 v = src[ui * n4 + j];
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        dst[j] = s;
    }
}

using encode_tiled_fn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                     const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                     CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
// cuTensorMapEncodeTiled, fetched from the driver through the runtime (the library does not link libcuda)
encode_tiled_fn encode_tiled() {
    static encode_tiled_fn fn = [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            ptr = nullptr;
        return reinterpret_cast<encode_tiled_fn>(ptr);
    }();
    return fn;
}

int units_per_file(long long rows) { return rows % (4 * RB) == 0 ? 4 : 1; }

}  // namespace

bool ccdc_map_cluster_fits(long long rows, long long d) {
    return rows >= RB && rows % RB == 0 && d % COLS_CTA == 0 && d / COLS_CTA <= MAX_CLUSTER &&
           ((d / COLS_CTA) & (d / COLS_CTA - 1)) == 0;
}

size_t ccdc_map_cluster_pieces_bytes(long long njobs, long long rows, long long d) {
    if (!ccdc_map_cluster_fits(rows, d)) return 0;
    return (size_t)njobs * units_per_file(rows) * d * 4;
}

int ccdc_map_cluster_launch(const ccdc_plan_s &P, const void *const *files_x, const void *const *files_y,
                            const void *w, long long rows, void *const *part, const long long *first_job,
                            void *pieces, int *status, void *stream) {
    const long long d = P.row_elems;
    if (!ccdc_map_cluster_fits(rows, d) || !encode_tiled()) return 1;
    static_assert(sizeof(ClusterParams) < 32 * 1024, "kernel parameters");
    ClusterParams cp;
    std::memset(&cp, 0, sizeof(cp));
    for (int k = 0; k < P.K; ++k) {
        cp.first_job[k + 1] = first_job[k + 1];
        const long long nfiles = first_job[k + 1] - first_job[k];
        if (nfiles == 0) continue;
        if (nfiles * rows > 0x7fffffffLL) return CCDC_ESIZE;            // TMA coordinates are ints
        // X of node k as (64 columns, files * rows, d / 64 chunks of 128 bytes); a box is a block's 32 chunks of 8 rows.
        // In shared memory a box is [chunk][row][128 bytes], so the 8 rows an ldmatrix reads lie in
        // consecutive 128-byte lines and the 128-byte swizzle spreads them over all banks.
        const cuuint64_t dims[3] = {64, (cuuint64_t)(nfiles * rows), (cuuint64_t)(d / 64)};
        const cuuint64_t strides[2] = {(cuuint64_t)d * 2, 128};
        const cuuint32_t box[3] = {64, RB, CHUNKS_CTA}, estr[3] = {1, 1, 1};
        if (encode_tiled()(&cp.tmap[k], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(files_x[k]), dims,
                           strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return 1;
        cp.y[k] = static_cast<const float *>(files_y[k]);
        cp.part[k] = static_cast<float *>(part[k]);
    }
    cp.w = static_cast<const uint16_t *>(w);
    cp.pieces = static_cast<float *>(pieces);
    cp.status = status;
    cp.njobs = first_job[P.K];
    cp.rows = rows;
    cp.d = d;
    cp.K = P.K;
    cp.UF = units_per_file(rows);
    if (cp.njobs == 0) return CCDC_OK;

    const int C = (int)(d / COLS_CTA);
    const size_t smem = (size_t)STAGES * STAGE_BYTES + 1024;
    cudaError_t e = cudaFuncSetAttribute(k_map_cluster, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return ccdc_internal_cuda_fail((int)e);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(THREADS, 1, 1);
    cfg.gridDim = dim3((unsigned)C, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int resident = 0;
    e = cudaOccupancyMaxActiveClusters(&resident, k_map_cluster, &cfg);
    if (e != cudaSuccess) { cudaGetLastError(); return 1; }
    if (resident < 1) return 1;
    const long long units = cp.njobs * cp.UF;
    cp.nclusters = (int)std::min<long long>(resident, units);
    // the files whose units fall into two or more shares (a share boundary inside the file)
    cp.nsplit = 0;
    for (int c = 1; c < cp.nclusters && cp.nsplit >= 0; ++c) {
        const long long ub = share_start(units, cp.nclusters, c);
        if (ub % cp.UF == 0) continue;
        const int job = (int)(ub / cp.UF);
        if (cp.nsplit > 0 && cp.split_jobs[cp.nsplit - 1] == job) continue;
        if (cp.nsplit == MAX_SPLIT) cp.nsplit = -1;
        else cp.split_jobs[cp.nsplit++] = job;
    }
    cfg.gridDim = dim3((unsigned)(cp.nclusters * C), 1, 1);
    e = cudaLaunchKernelEx(&cfg, k_map_cluster, cp);
    if (e != cudaSuccess) return ccdc_internal_cuda_fail((int)e);
    ccdc_internal_count_launch();
    if (cp.nsplit != 0) {
        const unsigned nblocks = cp.nsplit > 0 ? (unsigned)cp.nsplit : (unsigned)cp.njobs;
        k_map_combine<<<dim3(nblocks, 8), 256, 0, cfg.stream>>>(cp);
        ccdc_internal_count_launch();
        e = cudaGetLastError();
        if (e != cudaSuccess) return ccdc_internal_cuda_fail((int)e);
    }
    return CCDC_OK;
}
