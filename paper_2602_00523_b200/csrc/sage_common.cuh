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

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

inline int launch_status() { return cudaGetLastError() == cudaSuccess ? SAGE_OK : SAGE_ERR_CUDA; }

}  // namespace sage
