// Map phase of the linear-regression workload (Section III, "Map phase": node k
// maps every file it stores into Q intermediate values).  For file n the Q
// values are the Q contiguous slices of the partial gradient
//     g_n = X_n^T (X_n w - y_n),        X_n [rows][d] bf16, d = Q*B.
// Both products run on the tensor cores (mma.sync m16n8k16, bf16 operands, fp32
// accumulators).  The shape is matrix-vector, so the kernels are bound by the
// read of X_n; they are laid out so that every 16-byte load is coalesced and X_n
// never passes through shared memory:
//   pass 1  u = X w - y        A = 16 rows of X (k = columns), B = w in column 0
//   pass 2  g = X^T u          A = u split into three bf16 terms (rows 0..2),
//                              B = 16 rows x 8 columns of X, packed from four
//                              row vectors with byte permutes
// Every node maps its own copy of a file with the same code and the same fixed
// summation order, so the replicas are bit-identical (no atomics anywhere).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>

#include "ccdc_internal.h"

namespace {

// Files can be mapped in waves whose X stays in L2 between the two passes
// (CCDC_MAP_WAVE_MB > 0).  Measured on B200 that loses: grids of a wave are too
// small to saturate HBM (1.48 ms at 96 MB per wave against 0.92 ms for one wave
// over all 336 files of the K = 8 workload, where each pass streams X at the
// HBM rate).  0 = one wave.
#ifndef CCDC_MAP_WAVE_MB
#define CCDC_MAP_WAVE_MB 0
#endif
constexpr int MAP_THREADS = 256;                 // pass 1: 8 warps share 16 rows
constexpr int MAP_WARPS = MAP_THREADS / 32;
constexpr int GRAD_THREADS = 128;                // pass 2: 4 warps x 64 columns
constexpr int GRAD_WARPS = GRAD_THREADS / 32;
constexpr int GRAD_COLS = GRAD_WARPS * 64;

struct MapParams {
    const uint16_t *x[CCDC_MAX_K];      // node k: [local file][rows][d] bf16
    const float *y[CCDC_MAX_K];         // node k: [local file][rows]
    uint32_t *part[CCDC_MAX_K];         // node k: [local file][d] fp32 = [q][B]
    long long first_job[CCDC_MAX_K + 1];// jobs are (node, local file), node-major
    const uint16_t *w;                  // [d] bf16
    float *u;                           // [jobs][rows] residuals (workspace)
    long long job0, njobs;              // this wave
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

__device__ __forceinline__ int node_of_job(const MapParams &p, long long job) {
    int k = 0;
    while (k + 1 < p.K && job >= p.first_job[k + 1]) ++k;
    return k;
}

// ---- pass 1: u = X w - y for 16 rows of one file per block.
// The k index of the MMA is a free relabelling of the columns: thread (g, t)
// of a warp loads 8 consecutive columns of rows g and g+8 with one 16-byte load
// each and feeds them as k = 2t, 2t+1, 2t+8, 2t+9 of two MMAs; w is placed in
// column n = 0 of B with the same relabelling (lanes with g = 0), the other
// columns are zero.
__global__ void __launch_bounds__(MAP_THREADS)
k_map_residual(const __grid_constant__ MapParams p) {
    extern __shared__ __align__(16) uint32_t sh_w[];        // d/2 words: w as bf16 pairs
    __shared__ float sh_part[MAP_WARPS][16];
    const long long row_blocks = p.rows / 16;
    const long long job = p.job0 + blockIdx.x / row_blocks;
    const long long row0 = (blockIdx.x % row_blocks) * 16;
    const int k = node_of_job(p, job);
    const long long file = job - p.first_job[k];
    const uint16_t *X = p.x[k] + (file * p.rows + row0) * p.d;

    for (long long i = threadIdx.x; i < p.d / 8; i += MAP_THREADS)
        reinterpret_cast<uint4 *>(sh_w)[i] = __ldg(reinterpret_cast<const uint4 *>(p.w) + i);
    __syncthreads();

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int g = lane / 4, t = lane % 4;
    const long long cols_per_warp = p.d / MAP_WARPS;        // a multiple of 64
    const uint16_t *rowA = X + (long long)g * p.d;
    const uint16_t *rowB = X + (long long)(g + 8) * p.d;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (long long c0 = warp * cols_per_warp; c0 < (warp + 1) * cols_per_warp; c0 += 64) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const long long c = c0 + 32 * half + 8 * t;
            const uint4 va = __ldg(reinterpret_cast<const uint4 *>(rowA + c));
            const uint4 vb = __ldg(reinterpret_cast<const uint4 *>(rowB + c));
            uint4 wv = make_uint4(0u, 0u, 0u, 0u);
            if (g == 0) wv = *reinterpret_cast<const uint4 *>(sh_w + c / 2);
            mma_bf16(acc, va.x, vb.x, va.y, vb.y, wv.x, wv.y);
            mma_bf16(acc, va.z, vb.z, va.w, vb.w, wv.z, wv.w);
        }
    }
    // column n = 0 of the accumulator tile: thread (g, t = 0) holds rows g and g+8
    if (t == 0) {
        sh_part[warp][g] = acc[0];
        sh_part[warp][g + 8] = acc[2];
    }
    __syncthreads();
    if (threadIdx.x < 16) {
        float s = sh_part[0][threadIdx.x];
        for (int wv = 1; wv < MAP_WARPS; ++wv) s += sh_part[wv][threadIdx.x];   // fixed order
        const long long r = row0 + threadIdx.x;
        p.u[job * p.rows + r] = s - p.y[k][file * p.rows + r];
    }
}

// ---- pass 2: g = X^T u for GRAD_COLS columns of one file per block.
// A (16 x 16): row 0, 1, 2 = the three bf16 terms of u (u = hi + mid + lo to
// about 2^-25 relative), the other rows zero; k = 16 rows of X.  B (16 x 8):
// thread (g, t) supplies column n = g for k = 2t, 2t+1, 2t+8, 2t+9, i.e. one
// column of four rows.  It loads 8 columns of those four rows (16 bytes each)
// and serves eight MMAs, one per column of its octet, packing two rows into a
// register with a byte permute.  MMA e therefore produces, at n = g', column
// j0 + 8 g' + e.
__global__ void __launch_bounds__(GRAD_THREADS)
k_map_gradient(const __grid_constant__ MapParams p) {
    extern __shared__ __align__(16) uint32_t sh_u[];        // [3][rows/2] bf16 pairs: hi, mid, lo
    const long long col_blocks = (p.d + GRAD_COLS - 1) / GRAD_COLS;
    const long long job = p.job0 + blockIdx.x / col_blocks;
    const long long col0 = (blockIdx.x % col_blocks) * GRAD_COLS;
    const int k = node_of_job(p, job);
    const long long file = job - p.first_job[k];
    const uint16_t *X = p.x[k] + file * p.rows * p.d;
    const long long half_rows = p.rows / 2;

    for (long long i = threadIdx.x; i < half_rows; i += GRAD_THREADS) {
        uint32_t packed[3];
        float v[2] = {p.u[job * p.rows + 2 * i], p.u[job * p.rows + 2 * i + 1]};
        uint16_t term[3][2];
        for (int e = 0; e < 2; ++e) {
            float rest = v[e];
            for (int s = 0; s < 3; ++s) {
                const __nv_bfloat16 h = __float2bfloat16_rn(rest);
                term[s][e] = __bfloat16_as_ushort(h);
                rest = rest - __bfloat162float(h);          // exact in fp32
            }
        }
        for (int s = 0; s < 3; ++s) packed[s] = (uint32_t)term[s][0] | ((uint32_t)term[s][1] << 16);
        sh_u[i] = packed[0];
        sh_u[half_rows + i] = packed[1];
        sh_u[2 * half_rows + i] = packed[2];
    }
    __syncthreads();

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int g = lane / 4, t = lane % 4;
    const long long j0 = col0 + warp * 64;
    if (j0 >= p.d) return;
    const uint16_t *base = X + j0 + 8 * g;
    float acc[8][4];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e][0] = acc[e][1] = acc[e][2] = acc[e][3] = 0.f;

    for (long long i0 = 0; i0 < p.rows; i0 += 16) {
        const long long r0 = i0 + 2 * t;
        const uint4 v0 = __ldg(reinterpret_cast<const uint4 *>(base + r0 * p.d));
        const uint4 v1 = __ldg(reinterpret_cast<const uint4 *>(base + (r0 + 1) * p.d));
        const uint4 v2 = __ldg(reinterpret_cast<const uint4 *>(base + (r0 + 8) * p.d));
        const uint4 v3 = __ldg(reinterpret_cast<const uint4 *>(base + (r0 + 9) * p.d));
        uint32_t a0 = 0u, a2 = 0u;
        if (g < 3) {
            a0 = sh_u[g * half_rows + r0 / 2];
            a2 = sh_u[g * half_rows + (r0 + 8) / 2];
        }
        const uint32_t w0[4] = {v0.x, v0.y, v0.z, v0.w}, w1[4] = {v1.x, v1.y, v1.z, v1.w};
        const uint32_t w2[4] = {v2.x, v2.y, v2.z, v2.w}, w3[4] = {v3.x, v3.y, v3.z, v3.w};
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const uint32_t sel = (e & 1) ? 0x7632u : 0x5410u;       // high or low halves of both words
            const uint32_t b0 = __byte_perm(w0[e / 2], w1[e / 2], sel);
            const uint32_t b1 = __byte_perm(w2[e / 2], w3[e / 2], sel);
            mma_bf16(acc[e], a0, 0u, a2, 0u, b0, b1);
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

long long total_jobs(const ccdc_plan_s &P) {
    long long n = 0;
    for (int k = 0; k < P.K; ++k) n += P.nlocal[k] * P.b;
    return n;
}

}  // namespace

extern "C" {

size_t ccdc_map_workspace_bytes(const ccdc_plan_t *plan, long long rows) {
    if (!plan || rows <= 0) return 0;
    return (size_t)(total_jobs(*plan) * rows) * sizeof(float);
}

int ccdc_map(ccdc_plan_t *plan, const void *const *files_x, const void *const *files_y, const void *w,
             long long rows, void *const *part, void *workspace, void *stream) {
    if (!plan || !files_x || !files_y || !w || !part || !workspace) return CCDC_EINVAL;
    const ccdc_plan_s &P = *plan;
    if (P.dtype != CCDC_F32) return CCDC_ESTATE;
    const long long d = P.row_elems;
    if (rows < 16 || rows % 16 != 0 || rows > 4096 || d % 512 != 0 || d > 65536) return CCDC_ESIZE;
    MapParams mp;
    std::memset(&mp, 0, sizeof(mp));
    for (int k = 0; k < P.K; ++k) {
        mp.first_job[k + 1] = mp.first_job[k] + P.nlocal[k] * P.b;
        if (P.nlocal[k] == 0) continue;
        if (!files_x[k] || !files_y[k] || !part[k]) return CCDC_EINVAL;
        if ((reinterpret_cast<uintptr_t>(files_x[k]) | reinterpret_cast<uintptr_t>(part[k])) & 15u) return CCDC_EINVAL;
        if (reinterpret_cast<uintptr_t>(files_y[k]) & 3u) return CCDC_EINVAL;
        mp.x[k] = static_cast<const uint16_t *>(files_x[k]);
        mp.y[k] = static_cast<const float *>(files_y[k]);
        mp.part[k] = static_cast<uint32_t *>(part[k]);
    }
    if ((reinterpret_cast<uintptr_t>(w) & 15u) || (reinterpret_cast<uintptr_t>(workspace) & 15u)) return CCDC_EINVAL;
    mp.w = static_cast<const uint16_t *>(w);
    mp.u = static_cast<float *>(workspace);
    mp.rows = rows; mp.d = d; mp.K = P.K;
    const long long njobs = mp.first_job[P.K];
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const long long file_bytes = rows * d * 2;
    const long long wave = CCDC_MAP_WAVE_MB > 0 ? std::max(1LL, ((long long)CCDC_MAP_WAVE_MB << 20) / file_bytes)
                                                : std::max(1LL, njobs);
    const size_t smem1 = (size_t)d * 2, smem2 = (size_t)rows * 6;
    if (smem1 > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(k_map_residual, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1);
        if (e != cudaSuccess) return ccdc_internal_cuda_fail((int)e);
    }
    const long long col_blocks = (d + GRAD_COLS - 1) / GRAD_COLS;
    for (long long j0 = 0; j0 < njobs; j0 += wave) {
        mp.job0 = j0;
        mp.njobs = std::min(wave, njobs - j0);
        k_map_residual<<<(unsigned)(mp.njobs * (rows / 16)), MAP_THREADS, smem1, st>>>(mp);
        ccdc_internal_count_launch();
        k_map_gradient<<<(unsigned)(mp.njobs * col_blocks), GRAD_THREADS, smem2, st>>>(mp);
        ccdc_internal_count_launch();
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return ccdc_internal_cuda_fail((int)e);
    }
    return CCDC_OK;
}

}  // extern "C"
