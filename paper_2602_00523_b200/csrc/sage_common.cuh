// Shared device/host helpers of the SAGE hot-path kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sage.h"

namespace sage {

constexpr int kHeadDim = 128;
constexpr int kPageSize = 64;

// First data-dependent error wins; kernels keep going on safe values or return early.
__device__ __forceinline__ void report_status(int32_t* status, int code) {
    if (status != nullptr) atomicCAS(status, 0, code);
}

// Ancestor-or-self bitset of node i of a tree with n nodes (local parent indices).
// Returns 0 and sets *bad when the parent chain breaks the tree rules
// (root = node 0 with parent -1; every other node has 0 <= parent < index).
__device__ __forceinline__ uint64_t ancestor_bits(const int32_t* __restrict__ parent, int n, int i, bool* bad) {
    uint64_t a = 0;
    int cur = i;
    for (int it = 0; it < SAGE_MAX_NODES && cur >= 0; ++it) {
        a |= 1ull << cur;
        int par = parent[cur];
        if (cur == 0) {
            if (par != -1) *bad = true;
            break;
        }
        if (par < 0 || par >= cur) {
            *bad = true;
            break;
        }
        cur = par;
    }
    return a;
}

// Query rows per KV head (nodes x group size) of the largest well-formed tree of a batch; called by a
// whole warp, every lane gets the result.  sage_tree_attention launches more than one kernel when the
// host only knows an upper bound of the tree sizes (the nodes arrays' capacity); each kernel works this
// figure out for itself and only the one whose turn it is runs.
__device__ __forceinline__ int max_tree_rows(const int32_t* __restrict__ node_offsets, int batch, int sum_nodes, int G,
                                             int lane) {
    int mx = 0;
    for (int b0 = 0; b0 < batch; b0 += 32) {
        const int b = b0 + lane;
        if (b < batch) {
            const int n0 = node_offsets[b], N = node_offsets[b + 1] - n0;
            if (N >= 1 && N <= SAGE_MAX_NODES && n0 >= 0 && n0 + N <= sum_nodes) mx = max(mx, N * G);
        }
    }
    for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    return mx;
}
// select: 0 = the kernel runs whatever the trees look like; 1 = only for trees of one 128-row tile;
// 2 = only for two row tiles; 3 = only for more.
__device__ __forceinline__ bool schedule_selected(int select, int rows) {
    return select == 0 || (select == 1 && rows <= 128) || (select == 2 && rows > 128 && rows <= 256) ||
           (select == 3 && rows > 256);
}

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

inline int launch_status() { return cudaGetLastError() == cudaSuccess ? SAGE_OK : SAGE_ERR_CUDA; }

}  // namespace sage
