// Fused softmax entropy + top-k over vocabulary-sized fp32 rows (Eq. 4, Eq. 7-9)
// and the draft-token expansion gather.
//
// Pass 1 (logits_partial_kernel): grid = (chunks, rows).  Every CTA streams one
// contiguous chunk of one row once from HBM with 16-byte loads.  Each thread keeps
// online softmax moments (m, s = sum e^(x-m), t = sum (x-m) e^(x-m)) in fp32 over its
// few dozen elements; threads are merged in fp64.  Each warp keeps the K best
// (value, index) pairs of its elements as 64-bit keys, one per lane, sorted; an
// element is only looked at more closely when it reaches the warp's current K-th
// value.  Keys order by value (with -0 == +0) and then by lowest index, so every
// merge order gives the same answer.
// Pass 2 (logits_finalize_kernel): one warp per row merges the chunks' moments in
// fp64 and does a shuffle-based multi-way merge of the chunks' sorted candidate
// lists, then derives lse, full entropy, log-probs, top-k entropy and alpha.
#include <math.h>

#include <mutex>

#include "sage_common.cuh"

namespace sage {

constexpr int kPartialThreads = 256;
constexpr int kPartialWarps = kPartialThreads / 32;
constexpr int kMaxChunks = 32;

__device__ __forceinline__ uint32_t order_key(float x) {
    x += 0.0f;                                   // -0 -> +0
    const uint32_t u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_value(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
__device__ __forceinline__ uint64_t make_key(float x, int idx) {
    return ((uint64_t)order_key(x) << 32) | (uint32_t)(0xffffffffu - (uint32_t)idx);
}

// e^d for d <= 0 through the hardware 2^x (relative error about 2^-22): one multiply and one
// special-function instruction instead of the library routine's range reduction.  The moments
// built from it are merged in fp64; the entropy stays well inside its 1e-5 bound.
__device__ __forceinline__ float exp_neg(float d) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(d * 1.4426950408889634f));
    return y;
}

struct WarpQueue {
    uint64_t q;        // lane j < K: j-th best key so far (0 = empty)
    uint64_t kth;      // key in lane K-1 (same in all lanes)
    float thr;         // value of kth, -inf while the queue is not full
    int K;
    __device__ __forceinline__ void init(int k) { q = 0; kth = 0; thr = -INFINITY; K = k; }
    // Called by the whole warp; `want` marks lanes that hold a candidate (x, idx).
    __device__ __forceinline__ void offer(bool want, float x, int idx, int lane) {
        unsigned b = __ballot_sync(0xffffffffu, want);
        while (b) {
            const int src = __ffs(b) - 1;
            b &= b - 1;
            const uint64_t mine = make_key(x, idx);
            const uint64_t cand = __shfl_sync(0xffffffffu, mine, src);
            if (cand > kth) {
                const unsigned gt = __ballot_sync(0xffffffffu, q > cand);   // lanes >= K hold 0
                const int pos = __popc(gt);
                const uint64_t up = __shfl_up_sync(0xffffffffu, q, 1);
                if (lane < K && lane >= pos) q = (lane == pos) ? cand : up;
                kth = __shfl_sync(0xffffffffu, q, K - 1);
                thr = kth ? key_value((uint32_t)(kth >> 32)) : -INFINITY;
            }
        }
    }
};

struct PartialParams {
    const float* logits;
    int64_t row_stride;
    int vocab, chunk_len, n_chunks, K;
    double* stats;      // [rows][n_chunks][3]  (M, S, T)
    uint64_t* cand;     // [rows][n_chunks][SAGE_MAX_TOPK]
};

__global__ void __launch_bounds__(kPartialThreads) logits_partial_kernel(PartialParams p) {
    __shared__ float s_wmax[kPartialWarps];
    __shared__ double s_ws[kPartialWarps], s_wt[kPartialWarps];
    __shared__ uint64_t s_keys[kPartialWarps * SAGE_MAX_TOPK];
    const int chunk = blockIdx.x, row = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int begin = chunk * p.chunk_len;
    const int end = min(p.vocab, begin + p.chunk_len);
    const float* rowp = p.logits + (int64_t)row * p.row_stride;

    float m = -1e30f, s = 0.f, t = 0.f;
    WarpQueue wq;
    wq.init(p.K);

    // 16-byte loads: `begin` and row_stride are multiples of 4 elements.
    const int n4 = (end - begin) >> 2;
    const float4* src4 = reinterpret_cast<const float4*>(rowp + begin);
    // Four 16-byte loads are in flight per thread before the first is used: the chunk is short
    // (a few dozen elements per thread), so the pass is bound by load latency, not by bandwidth.
    for (int i0 = 0; i0 < n4; i0 += 4 * kPartialThreads) {
        float4 vv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * kPartialThreads + tid;
            vv[u] = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            if (i < n4) vv[u] = __ldcs(src4 + i);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * kPartialThreads + tid;
            const bool live = i < n4;
            const float4 v = vv[u];
            if (live) {
                const float m4 = fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w));
                if (m4 > m) {
                    const float c = expf(m - m4);
                    t = c * fmaf(m - m4, s, t);
                    s *= c;
                    m = m4;
                }
                const float d0 = v.x - m, d1 = v.y - m, d2 = v.z - m, d3 = v.w - m;
                const float e0 = exp_neg(d0), e1 = exp_neg(d1), e2 = exp_neg(d2), e3 = exp_neg(d3);
                s += (e0 + e1) + (e2 + e3);
                t += fmaf(d0, e0, d1 * e1) + fmaf(d2, e2, d3 * e3);
            }
            // A lane's largest component goes first: it lifts the queue's threshold, so that most of
            // the other components no longer qualify (matters while the queue is still filling).
            const float m4q = fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w));
            const bool hit = live && m4q >= wq.thr;
            if (__any_sync(0xffffffffu, hit)) {
                const int base = begin + 4 * i;
                const int top = (v.x == m4q) ? 0 : (v.y == m4q) ? 1 : (v.z == m4q) ? 2 : 3;   // lowest index on ties
                wq.offer(hit, m4q, base + top, lane);
                wq.offer(live && top != 0 && v.x >= wq.thr, v.x, base + 0, lane);
                wq.offer(live && top != 1 && v.y >= wq.thr, v.y, base + 1, lane);
                wq.offer(live && top != 2 && v.z >= wq.thr, v.z, base + 2, lane);
                wq.offer(live && top != 3 && v.w >= wq.thr, v.w, base + 3, lane);
            }
        }
    }
    // ragged tail of the last chunk (vocab % 4 elements)
    {
        const int i = begin + 4 * n4 + tid;
        const bool live = (tid < 4) && i < end;
        float x = -INFINITY;
        if (live) {
            x = rowp[i];
            if (x > m) {
                const float c = expf(m - x);
                t = c * fmaf(m - x, s, t);
                s *= c;
                m = x;
            }
            const float d = x - m, e = expf(d);
            s += e;
            t = fmaf(d, e, t);
        }
        if (warp == 0) wq.offer(live && x >= wq.thr, x, i, lane);
    }

    // ---- moments: block max, then rescale every thread's (s, t) in fp64
    float wm = m;
    for (int o = 16; o > 0; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, o));
    if (lane == 0) s_wmax[warp] = wm;
    if (lane < p.K) s_keys[warp * SAGE_MAX_TOPK + lane] = wq.q;
    else if (lane < SAGE_MAX_TOPK) s_keys[warp * SAGE_MAX_TOPK + lane] = 0;
    __syncthreads();
    float M = s_wmax[0];
#pragma unroll
    for (int w = 1; w < kPartialWarps; ++w) M = fmaxf(M, s_wmax[w]);
    double ds = 0.0, dt = 0.0;
    if (s > 0.f) {
        const double dm = (double)m - (double)M;
        const double c = exp(dm);
        ds = c * (double)s;
        dt = c * ((double)t + dm * (double)s);
    }
    for (int o = 16; o > 0; o >>= 1) {
        ds += __shfl_xor_sync(0xffffffffu, ds, o);
        dt += __shfl_xor_sync(0xffffffffu, dt, o);
    }
    if (lane == 0) { s_ws[warp] = ds; s_wt[warp] = dt; }
    __syncthreads();
    const size_t slot = (size_t)row * p.n_chunks + chunk;
    if (tid == 0) {
        double S = 0.0, T = 0.0;
        for (int w = 0; w < kPartialWarps; ++w) { S += s_ws[w]; T += s_wt[w]; }
        p.stats[slot * 3 + 0] = (double)M;
        p.stats[slot * 3 + 1] = S;
        p.stats[slot * 3 + 2] = T;
    }
    // ---- candidates: rank each of the warps' keys among all of them (keys are unique)
    if (tid < kPartialWarps * SAGE_MAX_TOPK) {
        const uint64_t mine = s_keys[tid];
        if (mine != 0) {
            int rank = 0;
            for (int j = 0; j < kPartialWarps * SAGE_MAX_TOPK; ++j) rank += (s_keys[j] > mine) ? 1 : 0;
            if (rank < p.K) p.cand[slot * SAGE_MAX_TOPK + rank] = mine;
        }
    }
    // slots past the number of elements in this chunk stay empty
    const int have = min(end - begin, p.K);
    if (tid >= have && tid < SAGE_MAX_TOPK) p.cand[slot * SAGE_MAX_TOPK + tid] = 0;
}

struct FinalizeParams {
    const double* stats;
    const uint64_t* cand;
    int rows, n_chunks, k, k_entropy, K;
    int32_t* topk_idx;
    float* topk_logprob;
    float* entropy_full;
    float* entropy_topk;
    float* alpha;
    float* lse;
};

__global__ void logits_finalize_kernel(FinalizeParams p) {
    const int warps = blockDim.x >> 5;
    const int row = blockIdx.x * warps + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= p.rows) return;
    const size_t base = (size_t)row * p.n_chunks;
    // moments
    double Mc = -INFINITY, Sc = 0.0, Tc = 0.0;
    if (lane < p.n_chunks) {
        Mc = p.stats[(base + lane) * 3 + 0];
        Sc = p.stats[(base + lane) * 3 + 1];
        Tc = p.stats[(base + lane) * 3 + 2];
    }
    double M = Mc;
    for (int o = 16; o > 0; o >>= 1) M = fmax(M, __shfl_xor_sync(0xffffffffu, M, o));
    double S = 0.0, T = 0.0;
    if (lane < p.n_chunks && Sc > 0.0) {
        const double dm = Mc - M, c = exp(dm);
        S = c * Sc;
        T = c * (Tc + dm * Sc);
    }
    for (int o = 16; o > 0; o >>= 1) {
        S += __shfl_xor_sync(0xffffffffu, S, o);
        T += __shfl_xor_sync(0xffffffffu, T, o);
    }
    const double lnS = log(S);
    const double lse = M + lnS;
    if (lane == 0) {
        if (p.lse) p.lse[row] = (float)lse;
        if (p.entropy_full) p.entropy_full[row] = (float)(lnS - T / S);
    }
    // multi-way merge of the chunks' sorted candidate lists: lane c holds the head of list c
    int head = 0;
    uint64_t cur = (lane < p.n_chunks) ? p.cand[(base + lane) * SAGE_MAX_TOPK] : 0;
    double v1 = 0.0, wsum = 0.0, wlog = 0.0;     // top-k entropy accumulators (lane-uniform)
    for (int j = 0; j < p.K; ++j) {
        uint64_t best = cur;
        for (int o = 16; o > 0; o >>= 1) {
            const uint64_t other = __shfl_xor_sync(0xffffffffu, best, o);
            best = other > best ? other : best;
        }
        if (best != 0 && cur == best) {          // keys are unique: exactly one lane advances
            ++head;
            cur = (head < SAGE_MAX_TOPK) ? p.cand[(base + lane) * SAGE_MAX_TOPK + head] : 0;
        }
        const double v = (double)key_value((uint32_t)(best >> 32));
        const int idx = (int)(0xffffffffu - (uint32_t)best);
        if (j < p.k && lane == 0) {
            p.topk_idx[(size_t)row * p.k + j] = best ? idx : -1;
            if (p.topk_logprob) p.topk_logprob[(size_t)row * p.k + j] = (float)(v - lse);
        }
        if (j < p.k_entropy && best != 0) {
            if (j == 0) v1 = v;
            const double d = v - v1, w = exp(d);  // w_j = P_j / P_1
            wsum += w;
            wlog += w * d;
        }
    }
    if (lane == 0 && (p.entropy_topk || p.alpha)) {
        // P~_j = w_j / wsum;  H = -sum P~ ln P~ = ln(wsum) - wlog / wsum
        const double H = log(wsum) - wlog / wsum;
        if (p.entropy_topk) p.entropy_topk[row] = (float)H;
        if (p.alpha) {
            double a = 1.0;
            if (p.k_entropy > 1) a = fmin(1.0, fmax(0.0, 1.0 - H / log((double)p.k_entropy)));
            p.alpha[row] = (float)a;
        }
    }
}

// draft_token[i] = topk_idx[row(parent(i))][rank(i)]  (Section 2.2 "Tree-based Drafting")
__global__ void expand_gather_kernel(const int32_t* __restrict__ topk_idx, int k, int rows,
                                     const int32_t* __restrict__ parent, const int32_t* __restrict__ rank,
                                     const int32_t* __restrict__ node_offsets, const int32_t* __restrict__ root_token,
                                     int32_t* __restrict__ draft_token, int32_t* status) {
    const int b = blockIdx.x;
    const int n0 = node_offsets[b];
    const int n = node_offsets[b + 1] - n0;
    if (n < 1 || n > SAGE_MAX_NODES || n0 < 0 || n0 + n > rows) {
        if (threadIdx.x == 0) report_status(status, SAGE_STATUS_BAD_TREE);
        return;
    }
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int par = parent[n0 + i];
        if (i == 0) {
            draft_token[n0] = root_token[b];
        } else {
            const int r = rank[n0 + i];
            if (par < 0 || par >= i || r < 0 || r >= k) {
                report_status(status, SAGE_STATUS_BAD_TREE);
                draft_token[n0 + i] = -1;
            } else {
                draft_token[n0 + i] = topk_idx[(size_t)(n0 + par) * k + r];
            }
        }
    }
}

static int pick_chunks(int rows, int vocab) {
    int c = (592 + rows - 1) / rows;                 // about four CTAs per SM
    const int max_by_len = (vocab + 4095) / 4096;    // keep chunks >= 4096 elements
    if (c > max_by_len) c = max_by_len;
    if (c > kMaxChunks) c = kMaxChunks;
    if (c < 1) c = 1;
    return c;
}

}  // namespace sage

using namespace sage;

extern "C" size_t sage_expand_topk_workspace_size(int rows, int vocab) {
    if (rows <= 0 || vocab <= 0) return 0;
    const size_t slots = (size_t)rows * pick_chunks(rows, vocab);
    return slots * (3 * sizeof(double) + SAGE_MAX_TOPK * sizeof(uint64_t));
}

extern "C" int sage_expand_topk(const float* logits, int rows, int vocab, int64_t row_stride, int k, int k_entropy,
                                int32_t* topk_idx, float* topk_logprob, float* entropy_full, float* entropy_topk,
                                float* alpha, float* lse, const int32_t* parent, const int32_t* rank,
                                const int32_t* node_offsets, int batch, const int32_t* root_token,
                                int32_t* draft_token, void* ws, size_t ws_bytes, int32_t* status, void* stream) {
    if (!logits || !topk_idx || rows < 0 || vocab < 1 || row_stride < vocab) return SAGE_ERR_INVALID_ARG;
    if (k < 1 || k_entropy < 1) return SAGE_ERR_INVALID_ARG;
    if (k > SAGE_MAX_TOPK || k_entropy > SAGE_MAX_TOPK) return SAGE_ERR_UNSUPPORTED;
    const int K = k > k_entropy ? k : k_entropy;
    if (K > vocab) return SAGE_ERR_INVALID_ARG;
    if (((uintptr_t)logits & 15) || (row_stride & 3)) return SAGE_ERR_UNSUPPORTED;
    if (draft_token && (!parent || !rank || !node_offsets || !root_token || batch < 0)) return SAGE_ERR_INVALID_ARG;
    if (rows == 0) return SAGE_OK;
    if (rows > 65535) return SAGE_ERR_UNSUPPORTED;
    const size_t need = sage_expand_topk_workspace_size(rows, vocab);
    if (!ws || ws_bytes < need || ((uintptr_t)ws & 15)) return SAGE_ERR_WORKSPACE;
    const int C = pick_chunks(rows, vocab);
    int chunk_len = (vocab + C - 1) / C;
    chunk_len = (chunk_len + 3) & ~3;
    double* stats = reinterpret_cast<double*>(ws);
    uint64_t* cand = reinterpret_cast<uint64_t*>(stats + (size_t)rows * C * 3);
    PartialParams pp{logits, row_stride, vocab, chunk_len, C, K, stats, cand};
    logits_partial_kernel<<<dim3(C, rows), kPartialThreads, 0, as_stream(stream)>>>(pp);
    FinalizeParams fp{stats, cand, rows, C, k, k_entropy, K, topk_idx, topk_logprob,
                      entropy_full, entropy_topk, alpha, lse};
    logits_finalize_kernel<<<(rows + 3) / 4, 128, 0, as_stream(stream)>>>(fp);
    if (draft_token && batch > 0)
        expand_gather_kernel<<<batch, 64, 0, as_stream(stream)>>>(topk_idx, k, rows, parent, rank, node_offsets,
                                                                  root_token, draft_token, status);
    return launch_status();
}

// ---------------------------------------------------------------------------
// sage_expand_topk_static: the same computation with the scratch memory built
// into the library instead of supplied by the caller.
// ---------------------------------------------------------------------------
namespace sage {

// Scratch of the static variant.  It is part of the library image: every GPU on which
// the library's kernels get loaded holds these bytes until the process exits.
__device__ __align__(256) static unsigned char g_static_scratch[SAGE_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;

// Device address of g_static_scratch on the current device (nullptr on failure).  In host
// code the array's name is only a handle for the runtime, not a device address, so the
// address is looked up once per device, with that device current, and remembered.
static void* static_scratch_address() {
    static std::mutex mu;
    static void* addr[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        addr[dev] = p;
    }
    return addr[dev];
}

}  // namespace sage

extern "C" int sage_expand_topk_static(const float* logits, int rows, int vocab, int64_t row_stride, int k,
                                       int k_entropy, int32_t* topk_idx, float* topk_logprob, float* entropy_full,
                                       float* entropy_topk, float* alpha, float* lse, const int32_t* parent,
                                       const int32_t* rank, const int32_t* node_offsets, int batch,
                                       const int32_t* root_token, int32_t* draft_token, int32_t* status,
                                       void* stream) {
    if (rows < 0 || vocab < 1) return SAGE_ERR_INVALID_ARG;
    if (rows > 0 && sage_expand_topk_workspace_size(rows, vocab) > (size_t)SAGE_STATIC_SCRATCH_BYTES)
        return SAGE_ERR_TOO_LARGE;
    void* scratch = nullptr;
    if (rows > 0) {
        scratch = static_scratch_address();
        if (scratch == nullptr) return SAGE_ERR_CUDA;
    }
    // Every scratch slot the finalize kernel reads is written by the partial kernel of the
    // same call, so nothing has to be cleared between calls.
    return sage_expand_topk(logits, rows, vocab, row_stride, k, k_entropy, topk_idx, topk_logprob, entropy_full,
                            entropy_topk, alpha, lse, parent, rank, node_offsets, batch, root_token, draft_token,
                            scratch, (size_t)SAGE_STATIC_SCRATCH_BYTES, status, stream);
}
