// The small reductions that follow the scoring pass.
//
// What the scoring pass leaves per unit (unit = prompt x layer x kv head; an item = one of the
// unit's `nchunk` chunks of keys; a piece = a run of one item's keys inside one segment):
//   part_z [U][P][Rpad]       per (piece, window row) z = sum exp2(x - m) over the piece's keys
//   item_m, item_z [U*nchunk][Rpad]   per (item, row) the reference exponent m all of the item's
//                              pieces share, and the sum of their z -- written by the kernels that
//                              fix one reference per item (score_fast.cuh, score_stream.cuh)
//   part_m [U][P][Rpad]       per (piece, row) reference -- written only by the exact kernel
//                              (score_tc.cuh), whose running maximum moves inside an item
//   redo   [U*nchunk]         1 for the items the exact kernel recomputed after the fast one
// An item is "exact" when every item is (`all_exact`: the exact kernel did all the work) or when
// its redo flag is set; its rows' statistics are then rebuilt from its pieces.
// row_stats_kernel, shot_mass_kernel, shot_score_from_mass_kernel, shot_score_from_tokens_kernel:
// fixed-order reductions of those partials, and of per-token importances.
#pragma once
#include "common.cuh"

namespace shotkv {

struct PartialView {
    const float* part_m;      // [U][P][Rpad]
    const float* part_z;      // [U][P][Rpad]
    const float* item_m;      // [U * nchunk][Rpad]
    const float* item_z;      // [U * nchunk][Rpad]
    const int* redo;          // [U * nchunk], or NULL
    const int* chunk_first;   // [B][cf_stride]: first piece of every item of a prompt; entry nchunk = number of pieces
    int cf_stride, nchunk, P, Rpad, all_exact;
};

__device__ __forceinline__ bool item_is_exact(const PartialView& v, int item) {
    return v.all_exact || (v.redo && v.redo[item]);
}
// (m, z) of two partial sums merged: z relative to the larger reference
__device__ __forceinline__ void merge_mz(float& m, float& z, float mq, float zq) {
    const float mn = fmaxf(m, mq);
    const float mu = mn == SHOTKV_NEG_INF ? 0.f : mn;
    z = z * ex2f(m - mu) + zq * ex2f(mq - mu);
    m = mn;
}
// Row r of unit u over all of its keys: m = max reference, z = sum exp2(x - m).  Items in index
// order, an exact item's pieces in index order: the result does not depend on scheduling.
__device__ __forceinline__ void row_stats_of(const PartialView& v, int u, int b, int r, float& m, float& z) {
    m = SHOTKV_NEG_INF;
    z = 0.f;
    const int* cf = v.chunk_first + (size_t)b * v.cf_stride;
    for (int j = 0; j < v.nchunk; ++j) {
        const int item = u * v.nchunk + j;
        if (item_is_exact(v, item)) {
            const float* pm = v.part_m + (size_t)u * v.P * v.Rpad + r;
            const float* pz = v.part_z + (size_t)u * v.P * v.Rpad + r;
            for (int q = cf[j]; q < cf[j + 1]; ++q) merge_mz(m, z, pm[(size_t)q * v.Rpad], pz[(size_t)q * v.Rpad]);
        } else {
            merge_mz(m, z, v.item_m[(size_t)item * v.Rpad + r], v.item_z[(size_t)item * v.Rpad + r]);
        }
    }
}

// Per (unit, row): m = max over the unit's keys, Z = sum exp2(x - m); stores m and 1/Z (0 for
// padding rows and rows without weight).
__global__ void row_stats_kernel(const PartialView v, int units_per_prompt, int R, float* __restrict__ row_m,
                                 float* __restrict__ row_invz) {
    const int u = blockIdx.x;
    for (int r = threadIdx.x; r < v.Rpad; r += blockDim.x) {
        float m = 0.f, z = 0.f;
        if (r < R) row_stats_of(v, u, u / units_per_prompt, r, m, z);   // padding rows carry no weight; their partials may be anything
        row_m[(size_t)u * v.Rpad + r] = (r < R && m != SHOTKV_NEG_INF) ? m : 0.f;
        row_invz[(size_t)u * v.Rpad + r] = (r < R && z > 0.f) ? 1.f / z : 0.f;
    }
}

// Per unit: the mass every row puts on every shot, normalised and summed over the rows:
//   unit_shot[u][i] = sum_r ( sum_{pieces q of shot i} z_q[r] * exp2(m_q[r] - m[r]) ) / Z[r]
// Phase 1, one thread per row: the row's (m, 1/Z) from the item statistics, left in shared
// memory.  Phase 2, one warp per piece: the lanes read the piece's z over the rows four at a
// time, weight them, and one shuffle reduction gives the piece's mass; the weight
// exp2(m_item[r] - m[r]) / Z[r] is the same for all pieces of an item and is formed once per
// item, so an ordinary piece costs one read of its z and eight multiply-adds per lane (an exact
// item's pieces carry their own references and pay one exp2 per row).  Phase 3 adds the pieces of
// each shot in index order.  piece_seg is ascending: 0 = tokens before the first shot, 1..S =
// shots, S+1 = the question, larger = list padding.  Shared memory: P + 2 * THREADS floats.
template <int THREADS>
__global__ void __launch_bounds__(THREADS) shot_mass_kernel(const PartialView v, const int* __restrict__ piece_seg, int R,
                                                           int L, int Hkv, int S, float* __restrict__ unit_shot) {
    constexpr int NW = THREADS / 32, NH = THREADS / 128;
    static_assert(THREADS == 128 || THREADS == 256, "one thread per padded window row");
    extern __shared__ __align__(16) float sm_mass[];
    float* row_m = sm_mass;                      // [THREADS]
    float* row_w = row_m + THREADS;              // [THREADS]  1/Z, 0 for rows without weight
    float* piece_mass = row_w + THREADS;         // [P]
    const int u = blockIdx.x;
    const int b = u / (L * Hkv);
    const int r = threadIdx.x, warp = r >> 5, lane = r & 31;
    const int* seg = piece_seg + (size_t)b * v.P;
    const int* cf = v.chunk_first + (size_t)b * v.cf_stride;
    const int nreal = cf[v.nchunk];              // pieces that are not list padding (they come first)
    {
        float m = SHOTKV_NEG_INF, z = 0.f;
        if (r < R) row_stats_of(v, u, b, r, m, z);
        row_m[r] = m == SHOTKV_NEG_INF ? 0.f : m;
        row_w[r] = (r < R && z > 0.f) ? 1.f / z : 0.f;
    }
    __syncthreads();
    // rows 4*lane .. 4*lane+3 (and the same 128 further on when there are 256 rows)
    float4 rm[NH], rw[NH];
#pragma unroll
    for (int h = 0; h < NH; ++h) {
        rm[h] = reinterpret_cast<const float4*>(row_m)[h * 32 + lane];
        rw[h] = reinterpret_cast<const float4*>(row_w)[h * 32 + lane];
    }
    const float* pm = v.part_m + (size_t)u * v.P * v.Rpad;
    const float* pz = v.part_z + (size_t)u * v.P * v.Rpad;
    for (int j = 0; j < v.nchunk; ++j) {
        const int item = u * v.nchunk + j;
        const bool exact = item_is_exact(v, item);
        float4 f[NH];                            // ordinary item: exp2(m_item - m) / Z of this lane's rows
        if (!exact) {
#pragma unroll
            for (int h = 0; h < NH; ++h) {
                const float4 mi = reinterpret_cast<const float4*>(v.item_m + (size_t)item * v.Rpad)[h * 32 + lane];
                // a row without weight (padding, or nothing but underflow) has w = 0 and gets factor 0
                f[h].x = rw[h].x > 0.f ? ex2f(mi.x - rm[h].x) * rw[h].x : 0.f;
                f[h].y = rw[h].y > 0.f ? ex2f(mi.y - rm[h].y) * rw[h].y : 0.f;
                f[h].z = rw[h].z > 0.f ? ex2f(mi.z - rm[h].z) * rw[h].z : 0.f;
                f[h].w = rw[h].w > 0.f ? ex2f(mi.w - rm[h].w) * rw[h].w : 0.f;
            }
        }
        for (int q = cf[j] + warp; q < cf[j + 1]; q += NW) {
            float a = 0.f;
#pragma unroll
            for (int h = 0; h < NH; ++h) {
                const float4 z4 = reinterpret_cast<const float4*>(pz + (size_t)q * v.Rpad)[h * 32 + lane];
                if (exact) {
                    const float4 m4 = reinterpret_cast<const float4*>(pm + (size_t)q * v.Rpad)[h * 32 + lane];
                    a += rw[h].x > 0.f ? z4.x * ex2f(m4.x - rm[h].x) * rw[h].x : 0.f;
                    a += rw[h].y > 0.f ? z4.y * ex2f(m4.y - rm[h].y) * rw[h].y : 0.f;
                    a += rw[h].z > 0.f ? z4.z * ex2f(m4.z - rm[h].z) * rw[h].z : 0.f;
                    a += rw[h].w > 0.f ? z4.w * ex2f(m4.w - rm[h].w) * rw[h].w : 0.f;
                } else {
                    a = fmaf(z4.x, f[h].x, a);
                    a = fmaf(z4.y, f[h].y, a);
                    a = fmaf(z4.z, f[h].z, a);
                    a = fmaf(z4.w, f[h].w, a);
                }
            }
            a = warp_sum(a);
            if (lane == 0) piece_mass[q] = a;
        }
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
