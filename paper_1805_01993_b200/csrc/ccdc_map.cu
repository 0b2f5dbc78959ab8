// Map phase of the linear-regression workload (Section III, "Map phase": node k
// maps every file it stores into Q intermediate values).  For file n the Q
// values are the Q contiguous slices of the partial gradient
//     g_n = X_n^T (X_n w - y_n),        X_n [rows][d] bf16, d = Q*B.
// Both products run on the tensor cores (mma.sync m16n8k16, bf16 operands, fp32
// accumulators).  The shape is matrix-vector, so the work is bound by the read
// of X_n; every 16-byte load is coalesced and X_n never passes through shared
// memory:
//   pass 1  u = X w - y        A = 16 rows of X (k = columns), B = w in column 0
//   pass 2  g = X^T u          A = u split into three bf16 terms (rows 0..2),
//                              B = 16 rows x 8 columns of X, packed from four
//                              row vectors with byte permutes
// Every node maps its own copy of a file with the same code and the same fixed
// summation order, so the replicas are bit-identical (no floating-point atomics).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>

#include "ccdc_internal.h"
#include "ccdc_map_cluster.h"

namespace {

#ifndef CCDC_MAP_BLOCKS_PER_SM
#define CCDC_MAP_BLOCKS_PER_SM 3     // resident blocks per SM: bounds the files in flight, i.e. the L2 footprint
#endif
#ifndef CCDC_MAP_MIN_BLOCKS
#define CCDC_MAP_MIN_BLOCKS 2        // register budget: 65536 / (256 * MIN_BLOCKS) per thread
#endif
#ifndef CCDC_MAP_DEPTH1
#define CCDC_MAP_DEPTH1 8            // pass 1: 64-column steps per trip (2 loads each)
#endif
#ifndef CCDC_MAP_DEPTH2
#define CCDC_MAP_DEPTH2 2            // pass 2: 16-row steps per trip (4 loads each)
#endif
#ifndef CCDC_MAP_LAG
#define CCDC_MAP_LAG 4               // pass 2 of file f is handed out after pass 1 of file f + LAG
#endif
constexpr int MAP_THREADS = 256;                 // 8 warps
constexpr int MAP_WARPS = MAP_THREADS / 32;
constexpr int GRAD_COLS = MAP_WARPS * 64;        // pass 2: columns per block
constexpr int WAIT_LIMIT = 1 << 20;              // polls of a file's pass-1 counter before giving up

struct MapParams {
    const uint16_t *x[CCDC_MAX_K];      // node k: [local file][rows][d] bf16
    const float *y[CCDC_MAX_K];         // node k: [local file][rows]
    uint32_t *part[CCDC_MAX_K];         // node k: [local file][d] fp32 = [q][B]
    long long first_job[CCDC_MAX_K + 1];// jobs are (node, local file), node-major
    const uint16_t *w;                  // [d] bf16
    float *u;                           // [jobs][rows] residuals (workspace)
    int *done;                          // [jobs] pass-1 blocks finished per job (workspace, zeroed per call)
    int *ticket;                        // next work item (workspace, zeroed per call)
    int *status;                        // set to 1 if a wait ran out (workspace, zeroed per call)
    long long njobs;
    long long rows, d;
    int K;
};

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// 16-byte read-only load with an L2 eviction policy: pass 1 asks L2 to keep X
// (evict last), pass 2 reads it for the last time (evict first)
__device__ __forceinline__ uint64_t l2_policy_keep() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint64_t l2_policy_drop() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint4 load_keep(const uint16_t *ptr, uint64_t policy) {
    uint4 v;
    asm volatile("ld.global.nc.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(ptr), "l"(policy));
    return v;
}

__device__ __forceinline__ int node_of_job(const MapParams &p, long long job) {
    int k = 0;
    while (k + 1 < p.K && job >= p.first_job[k + 1]) ++k;
    return k;
}

// ---- pass 1: u = X w - y for 16 rows of one file.
// Both the k index and the row index of the MMA are free relabellings.  A warp
// step covers 8 rows x 64 columns with two fully coalesced loads (each 4 rows x
// 128 bytes): thread (g, t) reads 16 bytes of row g/2 (and of row 4 + g/2) at
// column 32 (g%2) + 8 t.  MMA row m = g thus holds half (g%2) of row g/2, so w
// is placed in TWO columns of B: n = 0 the first 32 columns of the step, n = 1
// the second 32 (lanes with g = 0, 1), and D[m][m%2] is that half's dot
// product.  The 8 warps are 2 row groups x 4 column quarters; partial dots are
// added in a fixed order.
template <int QUARTERS>     // 64-column steps per loop trip: 2 * QUARTERS loads in flight per thread
__device__ __forceinline__ void residual_block(const MapParams &p, const uint32_t *sh_w, float (*sh_part)[16],
                                               long long job, long long row0) {
    const int k = node_of_job(p, job);
    const long long file = job - p.first_job[k];
    const uint16_t *X = p.x[k] + (file * p.rows + row0) * p.d;
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int g = lane / 4, t = lane % 4;
    const int row_group = warp & 1, quarter = warp >> 1;
    const long long cols_per_warp = p.d / 4;                // a multiple of 64
    const long long col_off = 32 * (g & 1) + 8 * t;
    const uint16_t *rowA = X + (long long)(row_group * 8 + g / 2) * p.d + col_off;
    const uint16_t *rowB = rowA + 4 * p.d;
    const uint64_t keep = l2_policy_keep();
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (long long c0 = quarter * cols_per_warp; c0 < (quarter + 1) * cols_per_warp; c0 += 64 * QUARTERS) {
        uint4 va[QUARTERS], vb[QUARTERS];
#pragma unroll
        for (int q = 0; q < QUARTERS; ++q) {         // all loads of the trip first
            va[q] = load_keep(rowA + c0 + 64 * q, keep);
            vb[q] = load_keep(rowB + c0 + 64 * q, keep);
        }
#pragma unroll
        for (int q = 0; q < QUARTERS; ++q) {
            uint4 wv = make_uint4(0u, 0u, 0u, 0u);
            if (g < 2) wv = *reinterpret_cast<const uint4 *>(sh_w + (c0 + 64 * q + 32 * g + 8 * t) / 2);
            mma_bf16(acc, va[q].x, vb[q].x, va[q].y, vb[q].y, wv.x, wv.y);
            mma_bf16(acc, va[q].z, vb[q].z, va[q].w, vb[q].w, wv.z, wv.w);
        }
    }
    // D[m][m%2]: lane (g, t = 0) holds columns 0, 1 of MMA rows g and g+8
    if (t == 0) {
        sh_part[warp][g] = (g & 1) ? acc[1] : acc[0];
        sh_part[warp][g + 8] = (g & 1) ? acc[3] : acc[2];
    }
    __syncthreads();
    if (threadIdx.x < 16) {
        const int rg = threadIdx.x / 8, rr = threadIdx.x % 8;           // row group, row inside it
        const int m0 = rr < 4 ? 2 * rr : 8 + 2 * (rr - 4);              // its two half-rows in the MMA tile
        float s = 0.f;
        for (int qt = 0; qt < 4; ++qt) {                                // fixed order
            const int wsrc = qt * 2 + rg;
            s += sh_part[wsrc][m0] + sh_part[wsrc][m0 + 1];
        }
        const long long r = row0 + threadIdx.x;
        p.u[job * p.rows + r] = s - p.y[k][file * p.rows + r];
        __threadfence();                    // the residuals are visible before the job's counter moves
    }
    __syncthreads();
    if (threadIdx.x == 0) atomicAdd(p.done + job, 1);
}

// ---- pass 2: g = X^T u for GRAD_COLS columns of one file.
// A (16 x 16): row 0, 1, 2 = the three bf16 terms of u (u = hi + mid + lo to
// about 2^-25 relative), the other rows zero; k = 16 rows of X.  B (16 x 8):
// thread (g, t) supplies column n = g for k = 2t, 2t+1, 2t+8, 2t+9, i.e. one
// column of four rows.  It loads 8 columns of those four rows (16 bytes each)
// and serves eight MMAs, one per column of its octet, packing two rows into a
// register with a byte permute.  MMA e therefore produces, at n = g', column
// j0 + 8 g' + e.
template <int STEPS>        // 16-row steps per loop trip: 4 * STEPS loads in flight per thread
__device__ __forceinline__ void gradient_block(const MapParams &p, uint32_t *sh_u, long long job, long long col0) {
    const int k = node_of_job(p, job);
    const long long file = job - p.first_job[k];
    const uint16_t *X = p.x[k] + file * p.rows * p.d;
    const long long half_rows = p.rows / 2;
    for (long long i = threadIdx.x; i < half_rows; i += MAP_THREADS) {
        // written by other blocks of this launch: read through L2, not the SM's L1
        const float2 v2 = __ldcg(reinterpret_cast<const float2 *>(p.u + job * p.rows) + i);
        const float v[2] = {v2.x, v2.y};
        uint16_t term[3][2];
        for (int e = 0; e < 2; ++e) {
            float rest = v[e];
            for (int s = 0; s < 3; ++s) {
                const __nv_bfloat16 h = __float2bfloat16_rn(rest);
                term[s][e] = __bfloat16_as_ushort(h);
                rest = rest - __bfloat162float(h);          // exact in fp32
            }
        }
        for (int s = 0; s < 3; ++s) sh_u[s * half_rows + i] = (uint32_t)term[s][0] | ((uint32_t)term[s][1] << 16);
    }
    __syncthreads();

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int g = lane / 4, t = lane % 4;
    const long long j0 = col0 + warp * 64;
    if (j0 < p.d) {
        const uint16_t *base = X + j0 + 8 * g;
        const uint64_t drop = l2_policy_drop();
        float acc[8][4];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e][0] = acc[e][1] = acc[e][2] = acc[e][3] = 0.f;
        for (long long i0 = 0; i0 < p.rows; i0 += 16 * STEPS) {
            uint4 v[STEPS][4];
#pragma unroll
            for (int h = 0; h < STEPS; ++h) {            // all loads of the trip first
                const long long r0 = i0 + 16 * h + 2 * t;
                v[h][0] = load_keep(base + r0 * p.d, drop);
                v[h][1] = load_keep(base + (r0 + 1) * p.d, drop);
                v[h][2] = load_keep(base + (r0 + 8) * p.d, drop);
                v[h][3] = load_keep(base + (r0 + 9) * p.d, drop);
            }
#pragma unroll
            for (int h = 0; h < STEPS; ++h) {
                const long long r0 = i0 + 16 * h + 2 * t;
                uint32_t a0 = 0u, a2 = 0u;
                if (g < 3) {
                    a0 = sh_u[g * half_rows + r0 / 2];
                    a2 = sh_u[g * half_rows + (r0 + 8) / 2];
                }
                const uint32_t w0[4] = {v[h][0].x, v[h][0].y, v[h][0].z, v[h][0].w};
                const uint32_t w1[4] = {v[h][1].x, v[h][1].y, v[h][1].z, v[h][1].w};
                const uint32_t w2[4] = {v[h][2].x, v[h][2].y, v[h][2].z, v[h][2].w};
                const uint32_t w3[4] = {v[h][3].x, v[h][3].y, v[h][3].z, v[h][3].w};
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const uint32_t sel = (e & 1) ? 0x7632u : 0x5410u;   // high or low halves of both words
                    const uint32_t b0 = __byte_perm(w0[e / 2], w1[e / 2], sel);
                    const uint32_t b1 = __byte_perm(w2[e / 2], w3[e / 2], sel);
                    mma_bf16(acc[e], a0, 0u, a2, 0u, b0, b1);
                }
            }
        }
        // rows 0, 1, 2 of the accumulator tiles live in lanes g = 0, 1, 2 (same t):
        // g = (hi + mid) + lo, then lanes g = 0 write 16 consecutive outputs
        uint32_t *out = p.part[k] + file * p.d;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const float hi = acc[e][c];
                const float mid = __shfl_down_sync(0xffffffffu, hi, 4);
                const float lo = __shfl_down_sync(0xffffffffu, hi, 8);
                acc[e][c] = (hi + mid) + lo;
            }
        }
        if (g == 0) {
            // column of acc[e][c] = j0 + 8 * (2t + c) + e
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                float4 lo4 = make_float4(acc[0][c], acc[1][c], acc[2][c], acc[3][c]);
                float4 hi4 = make_float4(acc[4][c], acc[5][c], acc[6][c], acc[7][c]);
                float *dst = reinterpret_cast<float *>(out) + j0 + 8 * (2 * t + c);
                *reinterpret_cast<float4 *>(dst) = lo4;
                *reinterpret_cast<float4 *>(dst + 4) = hi4;
            }
        }
    }
}

// ---- both passes in one launch, so that pass 2 finds the file in L2.
// Work items are handed out in order through an atomic ticket: per file, its
// n1 pass-1 blocks (16 rows each), then the n2 pass-2 blocks (512 columns each)
// of the file LAG places earlier.  With 148 x 3 blocks resident only a handful
// of files (a few tens of MB of X) are between their two passes at any time,
// so the second read of X is served by L2 and DRAM sees X once.
// A pass-2 item waits until the file's pass-1 counter is complete.  Those
// pass-1 items carry smaller tickets, so they were taken by blocks that are
// already running and that wait on nothing: the wait always ends.  It is
// bounded all the same; if it ever ran out the block records that in `status`
// and goes on (the file's output is then wrong and ccdc_map_status says so).
__global__ void __launch_bounds__(MAP_THREADS, CCDC_MAP_MIN_BLOCKS)
k_map(const __grid_constant__ MapParams p) {
    extern __shared__ __align__(16) uint32_t sh[];
    uint32_t *sh_w = sh;                        // d/2 words: w as bf16 pairs
    uint32_t *sh_u = sh + p.d / 2;              // 3 * rows/2 words: u as hi / mid / lo bf16 pairs
    __shared__ float sh_part[MAP_WARPS][16];
    __shared__ long long sh_ticket;

    for (long long i = threadIdx.x; i < p.d / 8; i += MAP_THREADS)
        reinterpret_cast<uint4 *>(sh_w)[i] = __ldg(reinterpret_cast<const uint4 *>(p.w) + i);

    const long long n1 = p.rows / 16, n2 = (p.d + GRAD_COLS - 1) / GRAD_COLS, per = n1 + n2;
    const long long total = (p.njobs + CCDC_MAP_LAG) * per;
    // deeper load pipelines when the shape divides evenly
    const bool deep1 = (p.d / 4) % (64 * CCDC_MAP_DEPTH1) == 0;
    const bool deep2 = p.rows % (16 * CCDC_MAP_DEPTH2) == 0;
    for (;;) {
        __syncthreads();                        // sh_ticket, sh_u and sh_part are free again
        if (threadIdx.x == 0) sh_ticket = atomicAdd(p.ticket, 1);
        __syncthreads();
        const long long tk = sh_ticket;
        if (tk >= total) break;
        const long long step = tk / per, slot = tk - step * per;
        if (slot < n1) {
            if (step < p.njobs) {
                if (deep1) residual_block<CCDC_MAP_DEPTH1>(p, sh_w, sh_part, step, slot * 16);
                else residual_block<1>(p, sh_w, sh_part, step, slot * 16);
            }
        } else {
            const long long job = step - CCDC_MAP_LAG;
            if (job < 0) continue;
            if (threadIdx.x == 0) {
                const volatile int *done = p.done + job;
                int polls = 0;
                while (*done < (int)n1) {
                    if (++polls > WAIT_LIMIT) { atomicExch(p.status, 1); break; }
                    __nanosleep(100);
                }
                __threadfence();
            }
            __syncthreads();
            if (deep2) gradient_block<CCDC_MAP_DEPTH2>(p, sh_u, job, (slot - n1) * GRAD_COLS);
            else gradient_block<1>(p, sh_u, job, (slot - n1) * GRAD_COLS);
        }
    }
}


const char *last_kernel = "";       // which kernel the last ccdc_map launched (reported, not synchronised)

long long total_jobs(const ccdc_plan_s &P) {
    long long n = 0;
    for (int k = 0; k < P.K; ++k) if (ccdc_plan_node_is_local(&P, k)) n += P.node_nfiles[k];
    return n;
}

// workspace layout: residuals [jobs][rows] fp32, then (256-byte aligned) the
// pass-1 counters [jobs], the ticket and the status word
size_t residual_bytes(long long jobs, long long rows) { return ((size_t)(jobs * rows) * 4 + 255) / 256 * 256; }
size_t control_bytes(long long jobs) { return ((size_t)(jobs + 2) * 4 + 255) / 256 * 256; }

// Which kernel maps a shape: the cluster kernel (X read once, staged by TMA) where it fits, unless
// the library was built with -DCCDC_MAP_USE_CLUSTER=0.
#ifndef CCDC_MAP_USE_CLUSTER
#define CCDC_MAP_USE_CLUSTER 1
#endif
size_t pieces_bytes(long long jobs, long long rows, long long d) {
    return CCDC_MAP_USE_CLUSTER ? ccdc_map_cluster_pieces_bytes(jobs, rows, d) : 0;
}

}  // namespace

extern "C" {

size_t ccdc_map_workspace_bytes(const ccdc_plan_t *plan, long long rows) {
    if (!plan || rows <= 0) return 0;
    const long long jobs = total_jobs(*plan);
    return residual_bytes(jobs, rows) + control_bytes(jobs) + pieces_bytes(jobs, rows, plan->row_elems);
}

int ccdc_map(ccdc_plan_t *plan, const void *const *files_x, const void *const *files_y, const void *w,
             long long rows, void *const *part, void *workspace, void *stream) {
    if (!plan || !files_x || !files_y || !w || !part || !workspace) return CCDC_EINVAL;
    const ccdc_plan_s &P = *plan;
    if (P.dtype != CCDC_F32 || P.compression_mode) return CCDC_ESTATE;
    const long long d = P.row_elems;
    if (rows < 16 || rows % 16 != 0 || rows > 4096 || d % 512 != 0 || d > 65536) return CCDC_ESIZE;
    MapParams mp;
    std::memset(&mp, 0, sizeof(mp));
    for (int k = 0; k < P.K; ++k) {
        const bool here = P.nlocal[k] > 0 && ccdc_plan_node_is_local(plan, k);
        mp.first_job[k + 1] = mp.first_job[k] + (here ? P.node_nfiles[k] : 0);
        if (!here) continue;
        if (!files_x[k] || !files_y[k] || !part[k]) return CCDC_EINVAL;
        if ((reinterpret_cast<uintptr_t>(files_x[k]) | reinterpret_cast<uintptr_t>(part[k])) & 15u) return CCDC_EINVAL;
        if (reinterpret_cast<uintptr_t>(files_y[k]) & 3u) return CCDC_EINVAL;
        mp.x[k] = static_cast<const uint16_t *>(files_x[k]);
        mp.y[k] = static_cast<const float *>(files_y[k]);
        mp.part[k] = static_cast<uint32_t *>(part[k]);
    }
    if ((reinterpret_cast<uintptr_t>(w) & 15u) || (reinterpret_cast<uintptr_t>(workspace) & 15u)) return CCDC_EINVAL;
    const long long njobs = mp.first_job[P.K];
    if (njobs * (rows / 16 + (d + GRAD_COLS - 1) / GRAD_COLS) > 0x3fffffffLL) return CCDC_ESIZE;   // tickets are ints
    mp.w = static_cast<const uint16_t *>(w);
    mp.u = static_cast<float *>(workspace);
    int *control = reinterpret_cast<int *>(static_cast<char *>(workspace) + residual_bytes(njobs, rows));
    mp.done = control;
    mp.ticket = control + njobs;
    mp.status = control + njobs + 1;
    mp.njobs = njobs; mp.rows = rows; mp.d = d; mp.K = P.K;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(control, 0, control_bytes(njobs), st);
    if (e != cudaSuccess) return ccdc_internal_cuda_fail((int)e);
#if CCDC_MAP_USE_CLUSTER
    if (ccdc_map_cluster_fits(rows, d)) {
        void *pieces = static_cast<char *>(workspace) + residual_bytes(njobs, rows) + control_bytes(njobs);
        const int rc = ccdc_map_cluster_launch(P, files_x, files_y, w, rows, part, mp.first_job, pieces, mp.status, stream);
        if (rc != 1) { last_kernel = "k_map_cluster"; return rc; }
    }
#endif
    int dev = 0, sms = 0, per_sm = 0;
    e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return ccdc_internal_cuda_fail((int)e);

    // loads through registers
    const size_t smem = (size_t)d * 2 + (size_t)rows * 6;
    if (smem > 32 * 1024) {
        e = cudaFuncSetAttribute(k_map, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return ccdc_internal_cuda_fail((int)e);
    }
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_map, MAP_THREADS, smem);
    if (e != cudaSuccess) return ccdc_internal_cuda_fail((int)e);
    per_sm = std::max(1, std::min(per_sm, CCDC_MAP_BLOCKS_PER_SM));
    last_kernel = "k_map";
    k_map<<<(unsigned)(sms * per_sm), MAP_THREADS, smem, st>>>(mp);
    ccdc_internal_count_launch();
    e = cudaGetLastError();
    return e == cudaSuccess ? CCDC_OK : ccdc_internal_cuda_fail((int)e);
}

const char *ccdc_map_last_kernel(void) { return last_kernel; }

int ccdc_map_status(const ccdc_plan_t *plan, long long rows, const void *workspace) {
    if (!plan || !workspace || rows <= 0) return CCDC_EINVAL;
    const long long jobs = total_jobs(*plan);
    const char *status = static_cast<const char *>(workspace) + residual_bytes(jobs, rows) + (size_t)(jobs + 1) * 4;
    int word = 0;
    cudaError_t e = cudaMemcpy(&word, status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return ccdc_internal_cuda_fail((int)e);
    return word == 0 ? CCDC_OK : CCDC_ESTATE;
}

int ccdc_job_host(ccdc_plan_t *plan, const void *const *host_x, const void *const *host_y, const void *host_w,
                  long long rows, void *host_out, void *const *dev_x, void *const *dev_y, void *dev_w,
                  void *const *dev_part, void *dev_coded, void *dev_out, void *map_workspace, void *dev_workspace,
                  void *stream) {
    if (!plan || !host_x || !host_y || !host_w || !host_out || !dev_x || !dev_y || !dev_w) return CCDC_EINVAL;
    if (rows <= 0) return CCDC_ESIZE;
    const ccdc_plan_s &P = *plan;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const long long d = P.row_elems;
    for (int k = 0; k < P.K; ++k) {
        if (!(P.nlocal[k] > 0 && ccdc_plan_node_is_local(plan, k))) continue;
        if (!host_x[k] || !host_y[k] || !dev_x[k] || !dev_y[k]) return CCDC_EINVAL;
        const size_t nrows = (size_t)P.node_nfiles[k] * (size_t)rows;
        cudaError_t e = cudaMemcpyAsync(dev_x[k], host_x[k], nrows * (size_t)d * 2, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(dev_y[k], host_y[k], nrows * 4, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return ccdc_internal_cuda_fail((int)e);
    }
    cudaError_t e = cudaMemcpyAsync(dev_w, host_w, (size_t)d * 2, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return ccdc_internal_cuda_fail((int)e);
    int rc = ccdc_map(plan, (const void *const *)dev_x, (const void *const *)dev_y, dev_w, rows, dev_part,
                      map_workspace, stream);
    if (rc != CCDC_OK) return rc;
    rc = ccdc_shuffle(plan, (const void *const *)dev_part, dev_coded, dev_out, dev_workspace, stream);
    if (rc != CCDC_OK) return rc;
    e = cudaMemcpyAsync(host_out, dev_out, ccdc_out_bytes(plan), cudaMemcpyDeviceToHost, st);
    return e == cudaSuccess ? CCDC_OK : ccdc_internal_cuda_fail((int)e);
}

}  // extern "C"
