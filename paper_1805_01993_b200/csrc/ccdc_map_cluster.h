// Cluster form of the Map kernel (ccdc_map_cluster.cu): internal interface used by ccdc_map.
#pragma once

#include <cstddef>

#include "ccdc_internal.h"

// shapes the cluster kernel serves: rows a multiple of 16, d = 2048 * {1, 2, 4, 8}
bool ccdc_map_cluster_fits(long long rows, long long d);
// workspace for the pieces of files that straddle two shares of the work; 0 if the shape does not fit
size_t ccdc_map_cluster_pieces_bytes(long long njobs, long long rows, long long d);
// Launches the Map on `stream`.  first_job[K+1]: node-major job offsets (0 files for nodes not mapped here).
// Returns CCDC_OK, a negative CCDC_* error, or 1 when this device or driver cannot run the kernel
// (no tensor-map encoder, no room for a cluster): the caller then uses the register kernel.
int ccdc_map_cluster_launch(const ccdc_plan_s &plan, const void *const *files_x, const void *const *files_y,
                            const void *w, long long rows, void *const *part, const long long *first_job,
                            void *pieces, int *status, void *stream);
