// Second pass of per-token importance, and the small reductions that follow the scoring pass.
//
// column_sum_mma_kernel: with every window row's final maximum and 1/Z known (row_stats_kernel),
// the logits are recomputed with warp-level MMA (mma.sync m16n8k16, bf16 in, fp32 accumulate),
// normalised and summed over the rows: token_importance[t] = sum_r alpha[r][t].  One CTA owns a
// unit's R = G*W window rows (padded to 128 or 256, Q held in registers as A fragments) and walks
// a list of key ranges; K tiles of 64 keys are staged in shared memory with cp.async (double
// buffered) and read with ldmatrix.
//
// row_stats_kernel, shot_mass_kernel, shot_score_from_mass_kernel: fixed-order reductions of the
// per-(piece, row) partials (m, z) written by the tensor-core scoring kernel.
#pragma once
#include "common.cuh"

namespace shotkv {

struct ScoreParams {
    const __nv_bfloat16* Q;   // [B][L][H][W][d]
    const __nv_bfloat16* K;   // [B][L][Hkv][N][d]
    const int2* pieces;       // [B][P] key ranges [lo, hi)
    int P, ppc;               // pieces per prompt, pieces per CTA
    int L, H, Hkv, N, W, G, R, Rpad;
    float scale_log2;         // log2(e)/sqrt(d)
    const float* row_m;       // [U][Rpad]      final row maxima (log2 domain)
    const float* row_invz;    // [U][Rpad]      1/Z per row (0 for padding rows)
    float* imp;               // [U][N]         out
};

constexpr int kTileKeys = 64;

template <int D, int MB>
constexpr int score_mma_smem_bytes() {
    return 128 * MB * D * 2 + 2 * kTileKeys * D * 2 + 8 * kTileKeys * 4;
}

template <int D, int MB>
__global__ void __launch_bounds__(256, (MB == 1 ? 2 : 1)) column_sum_mma_kernel(const ScoreParams p) {
    constexpr int ROWB = D * 2;
    constexpr int CH = D / 8;
    constexpr int KS = D / 16;
    constexpr int RP = 128 * MB;
    constexpr int TK = kTileKeys;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* sQ = smem;
    unsigned char* sK = smem + RP * ROWB;
    float* sCs = reinterpret_cast<float*>(sK + 2 * TK * ROWB);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t4 = lane & 3;
    const int u = blockIdx.y;
    const int bl = u / p.Hkv, hk = u - bl * p.Hkv;
    const int b = bl / p.L;
    const __nv_bfloat16* Qu = p.Q + ((size_t)bl * p.H + (size_t)hk * p.G) * p.W * D;
    const __nv_bfloat16* Ku = p.K + (size_t)u * p.N * D;

    for (int c = tid; c < RP * CH; c += 256) {
        const int row = c / CH, ch = c - row * CH;
        const int src_row = row < p.R ? row : p.R - 1;
        cp_async16(smem_u32(sQ) + swz<ROWB>(row, ch), Qu + (size_t)src_row * D + ch * 8, row < p.R ? 16 : 0);
    }
    cp_async_commit();
    cp_async_wait<0>();
    __syncthreads();

    uint32_t afrag[MB][KS][4];
#pragma unroll
    for (int mb = 0; mb < MB; ++mb)
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            const int row = mb * 128 + warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
            const int chunk = ks * 2 + (lane >> 4);
            ldmatrix_x4(afrag[mb][ks][0], afrag[mb][ks][1], afrag[mb][ks][2], afrag[mb][ks][3],
                        smem_u32(sQ) + swz<ROWB>(row, chunk));
        }

    // the two rows (g and g+8) this thread owns in each 16-row block: causal limit, statistics
    int plim[MB][2];
    float rm[MB][2], rinv[MB][2];
#pragma unroll
    for (int mb = 0; mb < MB; ++mb)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            const int r = mb * 128 + warp * 16 + g + hf * 8;
            plim[mb][hf] = r < p.R ? p.N - p.W + (r % p.W) : p.N - 1;
            rm[mb][hf] = p.row_m[(size_t)u * p.Rpad + r];
            rinv[mb][hf] = p.row_invz[(size_t)u * p.Rpad + r];
        }

    const int piece_begin = blockIdx.x * p.ppc;
    const int piece_end = min(piece_begin + p.ppc, p.P);
    for (int pi = piece_begin; pi < piece_end; ++pi) {
        const int2 pc = p.pieces[(size_t)b * p.P + pi];
        const int lo = pc.x, hi = pc.y;
        const int ntile = (hi - lo + TK - 1) / TK;
        auto load_tile = [&](int t) {
            const uint32_t dst = smem_u32(sK) + (t & 1) * TK * ROWB;
            const int key0 = lo + t * TK;
            for (int c = tid; c < TK * CH; c += 256) {
                const int row = c / CH, ch = c - row * CH;
                const int key = key0 + row;
                const bool ok = key < hi;
                cp_async16(dst + swz<ROWB>(row, ch), Ku + (size_t)(ok ? key : lo) * D + ch * 8, ok ? 16 : 0);
            }
            cp_async_commit();
        };

        if (ntile > 0) load_tile(0);
        for (int t = 0; t < ntile; ++t) {
            if (t + 1 < ntile) {
                load_tile(t + 1);
                cp_async_wait<1>();
            } else {
                cp_async_wait<0>();
            }
            __syncthreads();

            float acc[MB][8][4];
#pragma unroll
            for (int mb = 0; mb < MB; ++mb)
#pragma unroll
                for (int n = 0; n < 8; ++n) acc[mb][n][0] = acc[mb][n][1] = acc[mb][n][2] = acc[mb][n][3] = 0.f;

            const uint32_t kb = smem_u32(sK) + (t & 1) * TK * ROWB;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t bfr[8][2];
#pragma unroll
                for (int np = 0; np < 4; ++np) {
                    const int key = np * 16 + ((lane >> 4) << 3) + (lane & 7);
                    const int chunk = ks * 2 + ((lane >> 3) & 1);
                    ldmatrix_x4(bfr[2 * np][0], bfr[2 * np][1], bfr[2 * np + 1][0], bfr[2 * np + 1][1],
                                kb + swz<ROWB>(key, chunk));
                }
#pragma unroll
                for (int mb = 0; mb < MB; ++mb)
#pragma unroll
                    for (int n = 0; n < 8; ++n) mma_bf16_16816(acc[mb][n], afrag[mb][ks], bfr[n][0], bfr[n][1]);
            }

            const int key0 = lo + t * TK;
            // scale to the log2 domain and mask (beyond the piece, or after the row's own position)
#pragma unroll
            for (int mb = 0; mb < MB; ++mb)
#pragma unroll
                for (int n = 0; n < 8; ++n)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int kc = key0 + n * 8 + 2 * t4 + (e & 1);
                        const bool ok = kc < hi && kc <= plim[mb][e >> 1];
                        acc[mb][n][e] = ok ? acc[mb][n][e] * p.scale_log2 : SHOTKV_NEG_INF;
                    }

            {
#pragma unroll
                for (int n = 0; n < 8; ++n) {
                    float v0 = 0.f, v1 = 0.f;
#pragma unroll
                    for (int mb = 0; mb < MB; ++mb)
#pragma unroll
                        for (int hf = 0; hf < 2; ++hf) {
                            v0 += ex2f(acc[mb][n][2 * hf] - rm[mb][hf]) * rinv[mb][hf];
                            v1 += ex2f(acc[mb][n][2 * hf + 1] - rm[mb][hf]) * rinv[mb][hf];
                        }
#pragma unroll
                    for (int o = 4; o <= 16; o <<= 1) {
                        v0 += __shfl_xor_sync(0xffffffffu, v0, o);
                        v1 += __shfl_xor_sync(0xffffffffu, v1, o);
                    }
                    if (g == 0) {
                        sCs[warp * TK + n * 8 + 2 * t4] = v0;
                        sCs[warp * TK + n * 8 + 2 * t4 + 1] = v1;
                    }
                }
                __syncthreads();
                if (tid < TK) {
                    float s = 0.f;
#pragma unroll
                    for (int w = 0; w < 8; ++w) s += sCs[w * TK + tid];
                    const int key = key0 + tid;
                    if (key < hi) p.imp[(size_t)u * p.N + key] = s;
                }
            }
            __syncthreads();
        }
    }
}

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

// Score(s_i) from per-token importance: one CTA per (b, l, shot); fixed summation order.
__global__ void __launch_bounds__(128) shot_score_from_tokens_kernel(const float* __restrict__ imp,
                                                                    const int* __restrict__ off, int L, int Hkv, int N,
                                                                    int S, float* __restrict__ shot_scores) {
    __shared__ float red[4];
    const int i = blockIdx.x, bl = blockIdx.y;
    const int b = bl / L;
    const int lo = off[(size_t)b * (S + 1) + i], hi = off[(size_t)b * (S + 1) + i + 1];
    float a = 0.f;
    for (int h = 0; h < Hkv; ++h) {
        const float* row = imp + ((size_t)bl * Hkv + h) * N;
        for (int t = lo + threadIdx.x; t < hi; t += 128) a += row[t];
    }
    a = warp_sum(a);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = a;
    __syncthreads();
    if (threadIdx.x == 0) shot_scores[(size_t)bl * S + i] = (red[0] + red[1] + red[2] + red[3]) / (float)(hi - lo);
}

}  // namespace shotkv
