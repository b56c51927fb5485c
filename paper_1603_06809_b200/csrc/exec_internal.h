// What exec.cu offers to the other host-side files of the library (shard.cpp).
#pragma once
#include <functional>

#include "walk_tables.h"

// Launch shape of a register walk: words per lane (1..8) and blocks, for a walk whose slice count
// at `u` words per lane is slices_for(u).  `few_hops`: the longest hop list has at most three hops.
// *group: how many neighbouring slices a block takes at a time (WalkDev::group).
int bcast_internal_walk_shape(bool few_hops, const std::function<long long(int)> &slices_for, int P, int sm_count, int *u,
                              int *grid, int *group);

// Enqueue one register-walk kernel (traced if w.trace is set) on the current device.
int bcast_internal_launch_walk(const WalkDev &w, int u, int grid, void *const *rank_bufs, int P, void *cuda_stream);

// Argument checks shared by the executors: pointers non-NULL, 16-byte aligned, pairwise disjoint.
int bcast_internal_validate_bufs(void *const *rank_bufs, size_t P, uint64_t nbytes);

// Remember a failed CUDA call for bcast_last_cuda_error() and map it to a BCAST_ERR_* code.
int bcast_internal_cuda_failed(int cuda_error);
