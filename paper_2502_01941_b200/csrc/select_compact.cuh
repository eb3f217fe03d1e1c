// Whole-shot selection under the token budget and K/V row compaction.
#pragma once
#include "common.cuh"

namespace shotkv {

constexpr int kSelectThreads = 256;

// Exclusive prefix sum over n ints in shared memory, in place; returns the total.  All threads
// of the CTA must call it.  Each thread scans a contiguous slice, slices are combined serially
// through `tmp` (kSelectThreads ints): n is at most a few thousand, latency is irrelevant here.
__device__ inline int block_exclusive_scan(int* a, int n, int* tmp) {
    const int tid = threadIdx.x;
    const int per = (n + kSelectThreads - 1) / kSelectThreads;
    const int lo = min(tid * per, n), hi = min(lo + per, n);
    int s = 0;
    for (int i = lo; i < hi; ++i) s += a[i];
    tmp[tid] = s;
    __syncthreads();
    if (tid == 0) {
        int run = 0;
        for (int i = 0; i < kSelectThreads; ++i) {
            const int v = tmp[i];
            tmp[i] = run;
            run += v;
        }
        tmp[kSelectThreads] = run;
    }
    __syncthreads();
    int run = tmp[tid];
    for (int i = lo; i < hi; ++i) {
        const int v = a[i];
        a[i] = run;
        run += v;
    }
    __syncthreads();
    return tmp[kSelectThreads];
}

// One CTA per (b, l).  Ranks the S shots by (score descending, index ascending), keeps whole
// shots while they fit the budget left after the always-kept tokens, and writes the kept token
// positions in ascending order.
//   mode 0: the longest prefix of the ranking that fits;  mode 1: every shot that still fits.
// Shared memory: S floats + 3*S ints + (kSelectThreads+1) ints.
__global__ void __launch_bounds__(kSelectThreads) select_shots_kernel(
    const float* __restrict__ shot_scores, const int* __restrict__ off, int L, int N, int S, int budget_tokens,
    int mode, int Mcap, uint8_t* __restrict__ keep, int* __restrict__ kept_idx, int* __restrict__ kept_count) {
    extern __shared__ __align__(16) unsigned char sm[];
    float* sc = reinterpret_cast<float*>(sm);
    int* order = reinterpret_cast<int*>(sc + S);   // rank -> shot
    int* cum = order + S;                          // rank -> length, then scanned
    int* kl = cum + S;                             // shot -> kept length, then destination offset
    int* tmp = kl + S;
    const int bl = blockIdx.x, b = bl / L, tid = threadIdx.x;
    const int* o = off + (size_t)b * (S + 1);
    const int pre = o[0], qst = o[S];
    const int always = pre + (N - qst);
    const int shot_budget = budget_tokens - always;

    for (int i = tid; i < S; i += kSelectThreads) {
        const float v = shot_scores[(size_t)bl * S + i];
        sc[i] = v == v ? v : SHOTKV_NEG_INF;     // a NaN score ranks last instead of breaking the total order
    }
    __syncthreads();
    for (int i = tid; i < S; i += kSelectThreads) {
        const float v = sc[i];
        int rank = 0;
        for (int j = 0; j < S; ++j) {
            const float w = sc[j];
            rank += (w > v) || (w == v && j < i);
        }
        order[rank] = i;
        cum[rank] = o[i + 1] - o[i];
    }
    __syncthreads();
    if (mode == 0) {
        block_exclusive_scan(cum, S, tmp);
        for (int r = tid; r < S; r += kSelectThreads) {
            const int i = order[r];
            const int len = o[i + 1] - o[i];
            kl[i] = (cum[r] + len <= shot_budget) ? len : 0;
        }
    } else {
        if (tid == 0) {
            int used = 0;
            for (int r = 0; r < S; ++r) {
                const int i = order[r];
                const int len = cum[r];
                if (used + len <= shot_budget) {
                    kl[i] = len;
                    used += len;
                } else {
                    kl[i] = 0;
                }
            }
        }
    }
    __syncthreads();
    for (int i = tid; i < S; i += kSelectThreads) keep[(size_t)bl * S + i] = kl[i] > 0;
    __syncthreads();
    const int kept_shot_tokens = block_exclusive_scan(kl, S, tmp);
    const int total = always + kept_shot_tokens;
    int* out = kept_idx + (size_t)bl * Mcap;
    if (tid == 0) kept_count[bl] = total;
    for (int t = tid; t < pre && t < Mcap; t += kSelectThreads) out[t] = t;
    const int warp = tid >> 5, lane = tid & 31;
    for (int i = warp; i < S; i += kSelectThreads / 32) {
        if (keep[(size_t)bl * S + i]) {
            const int dst = pre + kl[i], lo = o[i], len = o[i + 1] - o[i];
            for (int t = lane; t < len; t += 32)
                if (dst + t < Mcap) out[dst + t] = lo + t;
        }
    }
    const int qdst = pre + kept_shot_tokens;
    for (int t = tid; t < N - qst; t += kSelectThreads)
        if (qdst + t < Mcap) out[qdst + t] = qst + t;
    for (int t = total + tid; t < Mcap; t += kSelectThreads) out[t] = -1;
}

// Row gather: Kc[u][j] = K[u][kept_idx[bl][j]], same for V.  Rows are D bf16 = D/8 16-byte
// vectors; consecutive lanes move consecutive vectors of a row, each thread keeps four
// independent loads in flight.  grid = (row blocks, Hkv, B*L).
template <int D>
__global__ void __launch_bounds__(256) compact_kv_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V,
                                                        const int* __restrict__ kept_idx,
                                                        const int* __restrict__ kept_count, int Hkv, int N, int Mcap,
                                                        uint4* __restrict__ Kc, uint4* __restrict__ Vc) {
    constexpr int VPR = D / 8;                 // 16-byte vectors per row
    constexpr int ROWS = 256 / VPR * 4;        // rows per CTA per pass
    const int bl = blockIdx.z, h = blockIdx.y;
    const int count = min(kept_count[bl], Mcap);
    const int row_in = threadIdx.x / VPR, v = threadIdx.x % VPR;
    const size_t u = (size_t)bl * Hkv + h;
    const uint4* Ku = K + u * N * VPR;
    const uint4* Vu = V + u * N * VPR;
    uint4* Kcu = Kc + u * Mcap * VPR;
    uint4* Vcu = Vc + u * Mcap * VPR;
    const int* idx = kept_idx + (size_t)bl * Mcap;
    for (int j0 = blockIdx.x * ROWS; j0 < count; j0 += gridDim.x * ROWS) {
        uint4 kk[4], vv[4];
        int src[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int j = j0 + q * (256 / VPR) + row_in;
            src[q] = j < count ? idx[j] : -1;
            if (src[q] >= N) src[q] = -1;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (src[q] >= 0) {
                kk[q] = __ldg(Ku + (size_t)src[q] * VPR + v);
                vv[q] = __ldg(Vu + (size_t)src[q] * VPR + v);
            }
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (src[q] >= 0) {
                const int j = j0 + q * (256 / VPR) + row_in;
                Kcu[(size_t)j * VPR + v] = kk[q];
                Vcu[(size_t)j * VPR + v] = vv[q];
            }
    }
}

}  // namespace shotkv
