// The small reductions that follow the scoring pass.
//
// row_stats_kernel, shot_mass_kernel, shot_score_from_mass_kernel, shot_score_from_tokens_kernel:
// fixed-order reductions of the per-(piece, row) partials (m, z) written by the tensor-core scoring
// kernels, and of per-token importances.
#pragma once
#include "common.cuh"

namespace shotkv {

// Per (unit, row): m = max over pieces, Z = sum z_p * exp2(m_p - m); stores m and 1/Z
// (0 for padding rows).  Fixed piece order, so the result does not depend on scheduling.
// Pieces whose segment id is above `last_seg` are list padding and are skipped.
__global__ void row_stats_kernel(const float* __restrict__ part_m, const float* __restrict__ part_z,
                                 const int* __restrict__ piece_seg, int units_per_prompt, int last_seg, int P, int R,
                                 int Rpad, float* __restrict__ row_m, float* __restrict__ row_invz) {
    const int u = blockIdx.x;
    const int* seg = piece_seg + (size_t)(u / units_per_prompt) * P;
    for (int r = threadIdx.x; r < Rpad; r += blockDim.x) {
        if (r >= R) {   // padding rows carry no weight; their partials may be anything
            row_m[(size_t)u * Rpad + r] = 0.f;
            row_invz[(size_t)u * Rpad + r] = 0.f;
            continue;
        }
        const float* pm = part_m + (size_t)u * P * Rpad + r;
        const float* pz = part_z + (size_t)u * P * Rpad + r;
        float m = SHOTKV_NEG_INF;
        for (int q = 0; q < P; ++q)
            if (seg[q] <= last_seg) m = fmaxf(m, pm[(size_t)q * Rpad]);
        float z = 0.f;
        for (int q = 0; q < P; ++q)
            if (seg[q] <= last_seg) z += pz[(size_t)q * Rpad] * ex2f(pm[(size_t)q * Rpad] - m);
        row_m[(size_t)u * Rpad + r] = m;
        row_invz[(size_t)u * Rpad + r] = z > 0.f ? 1.f / z : 0.f;
    }
}

// Per unit: the mass every row puts on every shot, normalised and summed over the rows:
//   unit_shot[u][i] = sum_r ( sum_{pieces q of shot i} z_q[r] * exp2(m_q[r] - m[r]) ) / Z[r]
// One thread per row.  Each thread first reduces its row's pieces to (m, 1/Z), then walks the
// pieces again and the rows of every piece are summed with warp shuffles into shared memory
// (no block barrier per piece); a last pass adds the warps' partials and the pieces of each shot
// in index order.  piece_seg is ascending: 0 = tokens before the first shot, 1..S = shots,
// S+1 = the question, larger = list padding.  Shared memory: P * (THREADS/32 + 1) floats.
template <int THREADS>
__global__ void __launch_bounds__(THREADS) shot_mass_kernel(const float* __restrict__ part_m,
                                                           const float* __restrict__ part_z,
                                                           const int* __restrict__ piece_seg, int P, int R, int Rpad,
                                                           int L, int Hkv, int S, float* __restrict__ unit_shot) {
    constexpr int NW = THREADS / 32;
    extern __shared__ float sm_mass[];          // [P][NW] warp partials, then [P] piece masses
    float* piece_mass = sm_mass + (size_t)P * NW;
    const int u = blockIdx.x;
    const int b = u / (L * Hkv);
    const int r = threadIdx.x, warp = r >> 5, lane = r & 31;
    const int* seg = piece_seg + (size_t)b * P;
    const float* pm = part_m + (size_t)u * P * Rpad + r;
    const float* pz = part_z + (size_t)u * P * Rpad + r;
    const bool live = r < R;
    int nreal = 0;                               // pieces that are not list padding (they come first)
    while (nreal < P && seg[nreal] <= S + 1) ++nreal;
    // one pass for (m, Z) with a running maximum, one pass for the masses
    float m = SHOTKV_NEG_INF, z = 0.f;
    if (live) {
#pragma unroll 8
        for (int q = 0; q < nreal; ++q) {
            const float mq = pm[(size_t)q * Rpad], zq = pz[(size_t)q * Rpad];
            const float mn = fmaxf(m, mq);
            const float mu = mn == SHOTKV_NEG_INF ? 0.f : mn;
            z = z * ex2f(m - mu) + zq * ex2f(mq - mu);
            m = mn;
        }
    }
    const float invz = (live && z > 0.f) ? 1.f / z : 0.f;
#pragma unroll 8
    for (int q = 0; q < nreal; ++q) {
        float a = live ? pz[(size_t)q * Rpad] * ex2f(pm[(size_t)q * Rpad] - m) * invz : 0.f;
        a = warp_sum(a);
        if (lane == 0) sm_mass[q * NW + warp] = a;
    }
    __syncthreads();
    for (int q = threadIdx.x; q < nreal; q += THREADS) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) s += sm_mass[q * NW + w];
        piece_mass[q] = s;
    }
    __syncthreads();
    // shot i owns the consecutive pieces with seg == i + 1; find them by binary search
    for (int i = threadIdx.x; i < S; i += THREADS) {
        int lo = 0, hi = nreal;
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (seg[mid] < i + 1) lo = mid + 1; else hi = mid;
        }
        float s = 0.f;
        for (int q = lo; q < nreal && seg[q] == i + 1; ++q) s += piece_mass[q];
        unit_shot[(size_t)u * S + i] = s;
    }
}

// Score(s_i) = (1/k_i) * sum over the kv heads of the unit masses (prefill score equation).
__global__ void shot_score_from_mass_kernel(const float* __restrict__ unit_shot, const int* __restrict__ off, int L,
                                            int Hkv, int S, float* __restrict__ shot_scores) {
    const int bl = blockIdx.x;
    const int b = bl / L;
    for (int i = threadIdx.x; i < S; i += blockDim.x) {
        float s = 0.f;
        for (int h = 0; h < Hkv; ++h) s += unit_shot[((size_t)bl * Hkv + h) * S + i];
        const int k = off[(size_t)b * (S + 1) + i + 1] - off[(size_t)b * (S + 1) + i];
        shot_scores[(size_t)bl * S + i] = s / (float)k;
    }
}

// Score(s_i) from per-token importance: one warp per (b, l, shot), eight shots per CTA; every
// lane sums a fixed subset of the shot's (kv head, token) pairs and the lanes are added by
// shuffles, so the order is fixed.  (One CTA per shot spent most of its time being launched once
// the units are sentence-sized and number in the thousands.)
constexpr int kShotsPerCta = 8;
__global__ void __launch_bounds__(32 * kShotsPerCta) shot_score_from_tokens_kernel(const float* __restrict__ imp,
                                                                                   const int* __restrict__ off, int L,
                                                                                   int Hkv, int N, int S,
                                                                                   float* __restrict__ shot_scores) {
    const int i = blockIdx.x * kShotsPerCta + (threadIdx.x >> 5), bl = blockIdx.y, lane = threadIdx.x & 31;
    if (i >= S) return;
    const int b = bl / L;
    const int lo = off[(size_t)b * (S + 1) + i], hi = off[(size_t)b * (S + 1) + i + 1];
    float a = 0.f;
    for (int h = 0; h < Hkv; ++h) {
        const float* row = imp + ((size_t)bl * Hkv + h) * N;
        for (int t = lo + lane; t < hi; t += 32) a += row[t];
    }
    a = warp_sum(a);
    if (lane == 0) shot_scores[(size_t)bl * S + i] = a / (float)(hi - lo);
}

}  // namespace shotkv
