// Internal interface of the bulk-copy pipeline kernels (ccdc_stream.cu).
#pragma once

#include <cuda_runtime.h>

#include "ccdc_internal.h"

// can this plan's fused encode / decode run as bulk-copy pipelines (alignment, table size, device)?
bool ccdc_stream_supported(const ccdc_plan_s &P);
// words of a segment one block of these kernels covers
long long ccdc_stream_tile_words();
// one launch each, asynchronous on `st`; the caller adds the partial sums when P.nchunk > 1
int ccdc_stream_decode(const ccdc_plan_s &P, const void *const *part, const void *coded, void *out, void *ws,
                       cudaStream_t st);
int ccdc_stream_encode(const ccdc_plan_s &P, const void *const *part, void *coded, cudaStream_t st);
