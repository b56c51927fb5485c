// Internal layout of a plan, shared by the planner (plan.cpp) and the executor (exec.cu).
#pragma once
#include <cstdint>
#include <vector>

#include "bcast.h"

struct bcast_device_state;   // defined in exec.cu; owns the device tables cached by a plan
struct bcast_static_image;   // defined in exec.cu; host image of the tables bcast_exec_static uses

struct bcast_plan {
    int P = 0, root = 0, variant = 0;
    int ranks_per_node = 0;                     // 0: no node awareness; else the node-aware broadcast of Section II
    int chunks = 0;                             // chunks the message is cut into: P, or the number of nodes
    int L = 0;                                  // scatter levels, ceil(log2 of the processes that scatter)
    uint64_t nbytes = 0, S = 0;                 // message bytes, scatter_size
    std::vector<bcast_xfer_t> xfers;            // canonical order: (phase, step, dst_rank)
    std::vector<int64_t> step_begin;            // CSR over xfers, L + (P-1) + 1 entries
    std::vector<uint64_t> bytes_sent[4], bytes_recv[4], msgs_sent[4], msgs_recv[4];   // [phase][rank]
    uint64_t total_bytes = 0;
    mutable bcast_device_state *dev = nullptr;  // created by the first execution
    mutable bcast_static_image *static_img = nullptr;   // created by the first bcast_exec_static (host memory only)
};

// exec.cu: frees the cached device tables of a plan (no-op when there are none)
void bcast_device_state_free(bcast_device_state *dev);
// exec.cu: frees the host image kept for bcast_exec_static (no-op when there is none)
void bcast_static_image_free(bcast_static_image *img);
