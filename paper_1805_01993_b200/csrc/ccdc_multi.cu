// Several GPUs: the two ways the shuffle shards (one process per GPU).
//
//  1. Value-dimension shards.  Every step of the scheme acts element by element
//     along a segment (Section IV-B: sums, XORs and cancellations of words at
//     equal positions), so GPU g of `world` can own the sub-range
//     [g*w, (g+1)*w), w = s/world, of EVERY segment of every packet and run the
//     whole scheme on it alone: an exact instance of the scheme with a shorter
//     value and no exchange between GPUs.  Here: the index map, and a copy
//     kernel between the full and the sharded layout.
//  2. Node shards with peer stores (ccdc_encode_fused_peers): every GPU's coded
//     buffer must be addressable from the others.  Here: buffers that can be
//     opened from another process (CUDA IPC), so that the encode kernel of one
//     rank stores straight into the buffers of the others.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstring>

#include "ccdc_internal.h"

namespace {

struct ShardShape {
    long long len, s, w, len_local, B_local;
};

int shard_shape(int K, int r, int Q, long long B, int rank, int world, ShardShape *out) {
    if (K < 2 || K > CCDC_MAX_K || r < 1 || r > K - 1 || Q < K || Q % K != 0 || B < 1) return CCDC_EINVAL;
    if (world < 1 || rank < 0 || rank >= world) return CCDC_EINVAL;
    const long long per = Q / K, len = per * B;
    if (len % r != 0) return CCDC_EINVAL;                   // equal segments without zero extension
    const long long s = len / r;
    if (s % world != 0) return CCDC_EINVAL;                 // equal sub-ranges
    const long long w = s / world, len_local = (long long)r * w;
    if (len_local % per != 0) return CCDC_EINVAL;           // the local packet is again Q/K values
    *out = {len, s, w, len_local, len_local / per};
    return CCDC_OK;
}

// dst/src: [rows][K][len] (full) and [rows][K][len_local] (local); one thread per local word
__global__ void __launch_bounds__(256)
k_value_shard(const uint32_t *__restrict__ src, uint32_t *__restrict__ dst, long long packets, long long len,
              long long s, long long w, long long len_local, int rank, int to_local) {
    const long long x = (long long)blockIdx.x * 256 + threadIdx.x;
    if (x >= packets * len_local) return;
    const long long pk = x / len_local, p = x - pk * len_local;
    const long long i = p / w, off = p - i * w;
    const long long full = pk * len + i * s + (long long)rank * w + off;
    if (to_local) dst[x] = src[full];
    else dst[full] = src[x];
}

}  // namespace

extern "C" {

int ccdc_value_shard(int K, int r, int Q, long long B, int rank, int world, long long *B_local) {
    ShardShape sh;
    const int rc = shard_shape(K, r, Q, B, rank, world, &sh);
    if (rc != CCDC_OK) return rc;
    if (B_local) *B_local = sh.B_local;
    return CCDC_OK;
}

long long ccdc_value_shard_position(int K, int r, int Q, long long B, int rank, int world, long long local_pos) {
    ShardShape sh;
    if (shard_shape(K, r, Q, B, rank, world, &sh) != CCDC_OK) return -1;
    if (local_pos < 0 || local_pos >= sh.len_local) return -1;
    const long long i = local_pos / sh.w;
    return i * sh.s + (long long)rank * sh.w + (local_pos - i * sh.w);
}

int ccdc_value_shard_copy(int K, int r, int Q, long long B, int rank, int world, int to_local, const void *src,
                          void *dst, long long rows, void *stream) {
    ShardShape sh;
    const int rc = shard_shape(K, r, Q, B, rank, world, &sh);
    if (rc != CCDC_OK) return rc;
    if (!src || !dst || rows < 0) return CCDC_EINVAL;
    if ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 3u) return CCDC_EINVAL;
    const long long packets = rows * K, todo = packets * sh.len_local;
    if (todo == 0) return CCDC_OK;
    const long long blocks = (todo + 255) / 256;
    if (blocks > 0x7fffffffLL) return CCDC_ESIZE;
    k_value_shard<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint32_t *>(src), static_cast<uint32_t *>(dst), packets, sh.len, sh.s, sh.w, sh.len_local, rank,
        to_local != 0);
    ccdc_internal_count_launch();
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? CCDC_OK : ccdc_internal_cuda_fail((int)e);
}

// ---- a job whose Map results sit in host memory once per file -------------
// Every batch of files is copied to the device once, into the partition of the first node that
// stores it, and from there to the other r-1 nodes that store it (device-to-device): the
// host-to-device traffic is N*Q*B words instead of r times that.
int ccdc_shuffle_host_files(ccdc_plan_t *plan, const void *host_values, void *host_out, void *const *dev_part,
                            void *dev_coded, void *dev_out, void *dev_workspace, void *stream) {
    if (!plan || !host_values || !host_out || !dev_part) return CCDC_EINVAL;
    const ccdc_plan_s &P = *plan;
    if (P.compression_mode || P.shard_world > 1) return CCDC_ESTATE;
    for (int k = 0; k < P.K; ++k)
        if (P.nlocal[k] > 0 && (!dev_part[k] || (reinterpret_cast<uintptr_t>(dev_part[k]) & 15u))) return CCDC_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the files of a batch are consecutive in the host array and in every holder's partition: one copy per
    // batch and holder
    const size_t batch_bytes = (size_t)P.b * (size_t)P.row_elems * 4;
    const char *src = static_cast<const char *>(host_values);
    for (long long p = 0; p < P.nbatch; ++p) {
        char *first = nullptr;
        for (int x = 0; x < P.r; ++x) {
            const int k = P.batch_nodes[(size_t)p * P.r + x];
            char *dst = static_cast<char *>(dev_part[k]) + (size_t)P.slot[(size_t)k * P.nbatch + p] * batch_bytes;
            const cudaError_t e =
                first ? cudaMemcpyAsync(dst, first, batch_bytes, cudaMemcpyDeviceToDevice, st)
                      : cudaMemcpyAsync(dst, src + (size_t)P.batch_file0[p] * (size_t)P.row_elems * 4, batch_bytes,
                                        cudaMemcpyHostToDevice, st);
            if (e != cudaSuccess) return ccdc_internal_cuda_fail((int)e);
            if (!first) first = dst;
        }
    }
    const int rc = ccdc_shuffle(plan, (const void *const *)dev_part, dev_coded, dev_out, dev_workspace, stream);
    if (rc != CCDC_OK) return rc;
    const cudaError_t e = cudaMemcpyAsync(host_out, dev_out, ccdc_out_bytes(plan), cudaMemcpyDeviceToHost, st);
    return e == cudaSuccess ? CCDC_OK : ccdc_internal_cuda_fail((int)e);
}

// ---- buffers another process can open -----------------------------------
static_assert(CCDC_PEER_HANDLE_BYTES >= sizeof(cudaIpcMemHandle_t), "handle size");

int ccdc_peer_buffer_create(size_t bytes, void **dev_ptr, void *handle_out) {
    if (!dev_ptr || !handle_out || bytes == 0) return CCDC_EINVAL;
    *dev_ptr = nullptr;
    void *p = nullptr;
    cudaError_t e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) {
        ccdc_internal_cuda_fail((int)e);
        return e == cudaErrorMemoryAllocation ? CCDC_ENOMEM : CCDC_ECUDA;
    }
    cudaIpcMemHandle_t h;
    e = cudaIpcGetMemHandle(&h, p);
    if (e != cudaSuccess) { cudaFree(p); return ccdc_internal_cuda_fail((int)e); }
    std::memset(handle_out, 0, CCDC_PEER_HANDLE_BYTES);
    std::memcpy(handle_out, &h, sizeof(h));
    *dev_ptr = p;
    return CCDC_OK;
}

int ccdc_peer_buffer_open(const void *handle, void **dev_ptr) {
    if (!handle || !dev_ptr) return CCDC_EINVAL;
    cudaIpcMemHandle_t h;
    std::memcpy(&h, handle, sizeof(h));
    void *p = nullptr;
    const cudaError_t e = cudaIpcOpenMemHandle(&p, h, cudaIpcMemLazyEnablePeerAccess);
    if (e != cudaSuccess) return ccdc_internal_cuda_fail((int)e);
    *dev_ptr = p;
    return CCDC_OK;
}

int ccdc_peer_buffer_close(void *dev_ptr) {
    if (!dev_ptr) return CCDC_EINVAL;
    const cudaError_t e = cudaIpcCloseMemHandle(dev_ptr);
    return e == cudaSuccess ? CCDC_OK : ccdc_internal_cuda_fail((int)e);
}

int ccdc_peer_buffer_destroy(void *dev_ptr) {
    if (!dev_ptr) return CCDC_EINVAL;
    const cudaError_t e = cudaFree(dev_ptr);
    return e == cudaSuccess ? CCDC_OK : ccdc_internal_cuda_fail((int)e);
}

int ccdc_peer_buffer_copy(void *dst, const void *src, size_t bytes, void *stream) {
    if (!dst || !src) return CCDC_EINVAL;
    const cudaError_t e = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDefault, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? CCDC_OK : ccdc_internal_cuda_fail((int)e);
}

}  // extern "C"
