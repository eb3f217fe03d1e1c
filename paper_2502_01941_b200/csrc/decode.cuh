// Decode phase: per-step attention-score accumulation over the decode-side entries and
// periodic top-k eviction.
#pragma once
#include "common.cuh"
#include "select_compact.cuh"

namespace shotkv {

struct DecodeParams {
    const __nv_bfloat16* q;       // [B][L][H][d]
    const __nv_bfloat16* k_new;   // [B][L][Hkv][d]
    const __nv_bfloat16* v_new;   // [B][L][Hkv][d]
    const __nv_bfloat16* Kc;      // [U][Mcap][d]
    const int* kept_count;        // [B*L]
    __nv_bfloat16* Kd;            // [U][Dcap][d]
    __nv_bfloat16* Vd;            // [U][Dcap][d]
    float* partial;               // [U][Dcap]
    int H, Hkv, G, Mcap, Dcap, n_old;
    float scale_log2;
    const __nv_bfloat16* Vc;      // [U][Mcap][d]   (attention-output variant only)
    float* out;                   // [B][L][H][d]   (attention-output variant only)
};

// One CTA per (sequence, layer, kv head).  Each warp takes 16 keys at a time straight from
// global memory: thread (g, t) of a warp reads 16 contiguous bytes of key rows g and g+8 per
// 32-dim block, which serve as the A fragments of two m16n8k16 MMAs whose B operand is the
// group's (up to 8) query rows held in registers with the same k-index permutation.  The logits
// of the decode entries are parked in shared memory until the softmax statistics over all keys
// (kept prefill keys + decode keys) are known.
template <int D>
__global__ void __launch_bounds__(256) decode_score_kernel(const DecodeParams p) {
    constexpr int NB = D / 32;     // 32-dim blocks
    constexpr int VPR = D / 8;     // 16-byte vectors per row
    extern __shared__ __align__(16) unsigned char dsm[];
    float* sdec = reinterpret_cast<float*>(dsm);             // [8][Dcap]
    float* sred = sdec + 8 * p.Dcap;                         // [8 warps][8 rows][2]
    float* sfin = sred + 8 * 8 * 2;                          // [8 rows][2]  (m, 1/Z)

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t4 = lane & 3;
    const int u = blockIdx.x;
    const int bl = u / p.Hkv, hk = u - bl * p.Hkv;
    const int M = min(p.kept_count[bl], p.Mcap);
    const int n = p.n_old + 1;
    const int Ktot = M + n;
    const uint4* Kc_u = reinterpret_cast<const uint4*>(p.Kc + (size_t)u * p.Mcap * D);
    uint4* Kd_u = reinterpret_cast<uint4*>(p.Kd + (size_t)u * p.Dcap * D);
    uint4* Vd_u = reinterpret_cast<uint4*>(p.Vd + (size_t)u * p.Dcap * D);
    const uint4* knew_u = reinterpret_cast<const uint4*>(p.k_new + (size_t)u * D);
    const uint4* vnew_u = reinterpret_cast<const uint4*>(p.v_new + (size_t)u * D);

    // append the new token's key and value as decode entry n_old
    if (tid < VPR) Kd_u[(size_t)p.n_old * VPR + tid] = knew_u[tid];
    else if (tid < 2 * VPR) Vd_u[(size_t)p.n_old * VPR + (tid - VPR)] = vnew_u[tid - VPR];

    // query rows of this group as B fragments (row g of the fragment = query head hk*G+g)
    uint4 qf[NB];
    {
        const uint4* qrow = reinterpret_cast<const uint4*>(p.q + ((size_t)bl * p.H + (size_t)hk * p.G + g) * D);
#pragma unroll
        for (int kb = 0; kb < NB; ++kb) qf[kb] = g < p.G ? qrow[kb * 4 + t4] : make_uint4(0, 0, 0, 0);
    }

    float m0 = SHOTKV_NEG_INF, m1 = SHOTKV_NEG_INF, z0 = 0.f, z1 = 0.f;   // query rows 2*t4, 2*t4+1
    for (int base = warp * 16; base < Ktot; base += 8 * 16) {
        const int ia = base + g, ib = base + g + 8;
        const bool va = ia < Ktot, vb = ib < Ktot;
        auto row_ptr = [&](int i, bool valid) -> const uint4* {
            if (!valid) return knew_u;                     // any readable row; the result is masked
            if (i < M) return Kc_u + (size_t)i * VPR;
            const int j = i - M;
            return j == p.n_old ? knew_u : Kd_u + (size_t)j * VPR;
        };
        const uint4* pa = row_ptr(ia, va);
        const uint4* pb = row_ptr(ib, vb);
        uint4 a_lo[NB], a_hi[NB];
#pragma unroll
        for (int kb = 0; kb < NB; ++kb) {
            a_lo[kb] = pa[kb * 4 + t4];
            a_hi[kb] = pb[kb * 4 + t4];
        }
        float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int kb = 0; kb < NB; ++kb) {
            const uint32_t f0[4] = {a_lo[kb].x, a_hi[kb].x, a_lo[kb].y, a_hi[kb].y};
            const uint32_t f1[4] = {a_lo[kb].z, a_hi[kb].z, a_lo[kb].w, a_hi[kb].w};
            mma_bf16_16816(c, f0, qf[kb].x, qf[kb].y);
            mma_bf16_16816(c, f1, qf[kb].z, qf[kb].w);
        }
        const float xa0 = va ? c[0] * p.scale_log2 : SHOTKV_NEG_INF;
        const float xa1 = va ? c[1] * p.scale_log2 : SHOTKV_NEG_INF;
        const float xb0 = vb ? c[2] * p.scale_log2 : SHOTKV_NEG_INF;
        const float xb1 = vb ? c[3] * p.scale_log2 : SHOTKV_NEG_INF;
        if (va && ia >= M) {
            sdec[(2 * t4) * p.Dcap + (ia - M)] = xa0;
            sdec[(2 * t4 + 1) * p.Dcap + (ia - M)] = xa1;
        }
        if (vb && ib >= M) {
            sdec[(2 * t4) * p.Dcap + (ib - M)] = xb0;
            sdec[(2 * t4 + 1) * p.Dcap + (ib - M)] = xb1;
        }
        {
            const float mn = fmaxf(m0, fmaxf(xa0, xb0));
            const float mu = mn == SHOTKV_NEG_INF ? 0.f : mn;
            z0 = z0 * ex2f(m0 - mu) + ex2f(xa0 - mu) + ex2f(xb0 - mu);
            m0 = mn;
        }
        {
            const float mn = fmaxf(m1, fmaxf(xa1, xb1));
            const float mu = mn == SHOTKV_NEG_INF ? 0.f : mn;
            z1 = z1 * ex2f(m1 - mu) + ex2f(xa1 - mu) + ex2f(xb1 - mu);
            m1 = mn;
        }
    }
    // combine the (m, z) pairs of the 8 lanes that share t4, then of the 8 warps
#pragma unroll
    for (int o = 4; o <= 16; o <<= 1) {
        const float om0 = __shfl_xor_sync(0xffffffffu, m0, o), oz0 = __shfl_xor_sync(0xffffffffu, z0, o);
        const float om1 = __shfl_xor_sync(0xffffffffu, m1, o), oz1 = __shfl_xor_sync(0xffffffffu, z1, o);
        {
            const float mn = fmaxf(m0, om0), mu = mn == SHOTKV_NEG_INF ? 0.f : mn;
            z0 = z0 * ex2f(m0 - mu) + oz0 * ex2f(om0 - mu);
            m0 = mn;
        }
        {
            const float mn = fmaxf(m1, om1), mu = mn == SHOTKV_NEG_INF ? 0.f : mn;
            z1 = z1 * ex2f(m1 - mu) + oz1 * ex2f(om1 - mu);
            m1 = mn;
        }
    }
    if (g == 0) {
        sred[(warp * 8 + 2 * t4) * 2 + 0] = m0;
        sred[(warp * 8 + 2 * t4) * 2 + 1] = z0;
        sred[(warp * 8 + 2 * t4 + 1) * 2 + 0] = m1;
        sred[(warp * 8 + 2 * t4 + 1) * 2 + 1] = z1;
    }
    __syncthreads();
    if (tid < 8) {
        float m = SHOTKV_NEG_INF;
        for (int w = 0; w < 8; ++w) m = fmaxf(m, sred[(w * 8 + tid) * 2]);
        float z = 0.f;
        for (int w = 0; w < 8; ++w) z += sred[(w * 8 + tid) * 2 + 1] * ex2f(sred[(w * 8 + tid) * 2] - m);
        sfin[tid * 2] = m;
        sfin[tid * 2 + 1] = z > 0.f ? 1.f / z : 0.f;
    }
    __syncthreads();
    for (int j = tid; j < n; j += 256) {
        float s = 0.f;
        for (int r = 0; r < p.G; ++r) s += ex2f(sdec[r * p.Dcap + j] - sfin[r * 2]) * sfin[r * 2 + 1];
        p.partial[(size_t)u * p.Dcap + j] = s;
    }
}

// The same step with the attention output fused in: o_h = sum_t alpha_{t,h} v_t over the kept
// prefill entries and the decode entries, with the very weights the decoding score sums, so that
// scoring adds no pass over K to a decode step that has to read K and V anyway.  Per 16-key
// block a warp computes the logits as above, keeps a warp-wide running maximum per query row,
// shares the block's weights P (16 keys x 8 rows) through shared memory, and accumulates
// O[row][dims] += P[key][row] * V[key][dims] with every lane owning D/32 dimensions of all QR
// query rows.  The value rows are requested before the softmax arithmetic so that their latency
// overlaps it.  The eight warps' (m, z, O) are merged at the end in warp order.
template <int D, int QR>
__global__ void __launch_bounds__(256) decode_attend_kernel(const DecodeParams p) {
    constexpr int NB = D / 32;     // 32-dim blocks
    constexpr int VPR = D / 8;     // 16-byte vectors per row
    constexpr int DPT = D / 32;    // dimensions of a value row per lane (4 or 2)
    extern __shared__ __align__(16) unsigned char dsm[];
    float* sdec = reinterpret_cast<float*>(dsm);             // [8][Dcap]
    float* sred = sdec + 8 * p.Dcap;                         // [8 warps][8 rows][2]
    float* sfin = sred + 8 * 8 * 2;                          // [8 rows][2]  (m, 1/Z)
    float* sP = sfin + 16;                                   // [8 warps][16 keys + 1][8 rows]; row 16 = rescale factors
    float* sO = sP + 8 * 17 * 8;                             // [8 warps][QR][D]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t4 = lane & 3;
    const int u = blockIdx.x;
    const int bl = u / p.Hkv, hk = u - bl * p.Hkv;
    const int M = min(p.kept_count[bl], p.Mcap);
    const int n = p.n_old + 1;
    const int Ktot = M + n;
    const uint4* Kc_u = reinterpret_cast<const uint4*>(p.Kc + (size_t)u * p.Mcap * D);
    uint4* Kd_u = reinterpret_cast<uint4*>(p.Kd + (size_t)u * p.Dcap * D);
    uint4* Vd_u = reinterpret_cast<uint4*>(p.Vd + (size_t)u * p.Dcap * D);
    const uint4* knew_u = reinterpret_cast<const uint4*>(p.k_new + (size_t)u * D);
    const uint4* vnew_u = reinterpret_cast<const uint4*>(p.v_new + (size_t)u * D);
    const __nv_bfloat16* Vc_u = p.Vc + (size_t)u * p.Mcap * D;
    const __nv_bfloat16* Vd_e = p.Vd + (size_t)u * p.Dcap * D;
    const __nv_bfloat16* vnew_e = p.v_new + (size_t)u * D;

    // append the new token's key and value as decode entry n_old
    if (tid < VPR) Kd_u[(size_t)p.n_old * VPR + tid] = knew_u[tid];
    else if (tid < 2 * VPR) Vd_u[(size_t)p.n_old * VPR + (tid - VPR)] = vnew_u[tid - VPR];

    uint4 qf[NB];
    {
        const uint4* qrow = reinterpret_cast<const uint4*>(p.q + ((size_t)bl * p.H + (size_t)hk * p.G + g) * D);
#pragma unroll
        for (int kb = 0; kb < NB; ++kb) qf[kb] = g < p.G ? qrow[kb * 4 + t4] : make_uint4(0, 0, 0, 0);
    }

    float* sPw = sP + warp * 17 * 8;
    float O[QR][DPT];
#pragma unroll
    for (int r = 0; r < QR; ++r)
#pragma unroll
        for (int j = 0; j < DPT; ++j) O[r][j] = 0.f;
    // running maximum of query rows 2*t4 and 2*t4+1 over this warp's keys (the same in the 8 lanes
    // that share t4); z0, z1: this lane's part of the row sums relative to it
    float m0 = SHOTKV_NEG_INF, m1 = SHOTKV_NEG_INF, z0 = 0.f, z1 = 0.f;
    for (int base = warp * 16; base < Ktot; base += 8 * 16) {
        const int ia = base + g, ib = base + g + 8;
        const bool va = ia < Ktot, vb = ib < Ktot;
        auto row_ptr = [&](int i, bool valid) -> const uint4* {
            if (!valid) return knew_u;                     // any readable row; the result is masked
            if (i < M) return Kc_u + (size_t)i * VPR;
            const int j = i - M;
            return j == p.n_old ? knew_u : Kd_u + (size_t)j * VPR;
        };
        const uint4* pa = row_ptr(ia, va);
        const uint4* pb = row_ptr(ib, vb);
        uint4 a_lo[NB], a_hi[NB];
#pragma unroll
        for (int kb = 0; kb < NB; ++kb) {
            a_lo[kb] = pa[kb * 4 + t4];
            a_hi[kb] = pb[kb * 4 + t4];
        }
        // this lane's D/32 dimensions of the block's 16 value rows (rows past the end: zeros)
        uint32_t vraw[16][DPT / 2];
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            const int i = base + kk;
            const __nv_bfloat16* vr = i < M ? Vc_u + (size_t)i * D : (i - M == p.n_old ? vnew_e : Vd_e + (size_t)(i - M) * D);
            if (i < Ktot) {
                if (DPT == 4) {
                    const uint2 t = *reinterpret_cast<const uint2*>(vr + lane * 4);
                    vraw[kk][0] = t.x;
                    vraw[kk][DPT / 2 - 1] = t.y;
                } else {
                    vraw[kk][0] = *reinterpret_cast<const uint32_t*>(vr + lane * 2);
                }
            } else {
#pragma unroll
                for (int j = 0; j < DPT / 2; ++j) vraw[kk][j] = 0u;
            }
        }
        float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int kb = 0; kb < NB; ++kb) {
            const uint32_t f0[4] = {a_lo[kb].x, a_hi[kb].x, a_lo[kb].y, a_hi[kb].y};
            const uint32_t f1[4] = {a_lo[kb].z, a_hi[kb].z, a_lo[kb].w, a_hi[kb].w};
            mma_bf16_16816(c, f0, qf[kb].x, qf[kb].y);
            mma_bf16_16816(c, f1, qf[kb].z, qf[kb].w);
        }
        const float xa0 = va ? c[0] * p.scale_log2 : SHOTKV_NEG_INF;
        const float xa1 = va ? c[1] * p.scale_log2 : SHOTKV_NEG_INF;
        const float xb0 = vb ? c[2] * p.scale_log2 : SHOTKV_NEG_INF;
        const float xb1 = vb ? c[3] * p.scale_log2 : SHOTKV_NEG_INF;
        if (va && ia >= M) {
            sdec[(2 * t4) * p.Dcap + (ia - M)] = xa0;
            sdec[(2 * t4 + 1) * p.Dcap + (ia - M)] = xa1;
        }
        if (vb && ib >= M) {
            sdec[(2 * t4) * p.Dcap + (ib - M)] = xb0;
            sdec[(2 * t4 + 1) * p.Dcap + (ib - M)] = xb1;
        }
        // block maximum per query row over the 16 keys (lanes that share t4)
        float bm0 = fmaxf(xa0, xb0), bm1 = fmaxf(xa1, xb1);
#pragma unroll
        for (int o = 4; o <= 16; o <<= 1) {
            bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, o));
            bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, o));
        }
        const float mn0 = fmaxf(m0, bm0), mn1 = fmaxf(m1, bm1);
        const float mu0 = mn0 == SHOTKV_NEG_INF ? 0.f : mn0, mu1 = mn1 == SHOTKV_NEG_INF ? 0.f : mn1;
        const float al0 = ex2f(m0 - mu0), al1 = ex2f(m1 - mu1);         // rescale of what was summed so far
        const float pa0 = ex2f(xa0 - mu0), pb0 = ex2f(xb0 - mu0), pa1 = ex2f(xa1 - mu1), pb1 = ex2f(xb1 - mu1);
        z0 = z0 * al0 + pa0 + pb0;
        z1 = z1 * al1 + pa1 + pb1;
        const bool changed = __any_sync(0xffffffffu, mn0 != m0 || mn1 != m1);
        m0 = mn0;
        m1 = mn1;
        __syncwarp();                                      // the previous block's weights have been read
        sPw[g * 8 + 2 * t4] = pa0;
        sPw[g * 8 + 2 * t4 + 1] = pa1;
        sPw[(g + 8) * 8 + 2 * t4] = pb0;
        sPw[(g + 8) * 8 + 2 * t4 + 1] = pb1;
        if (g == 0) {
            sPw[16 * 8 + 2 * t4] = al0;
            sPw[16 * 8 + 2 * t4 + 1] = al1;
        }
        __syncwarp();
        if (changed) {
#pragma unroll
            for (int r = 0; r < QR; ++r) {
                const float al = sPw[16 * 8 + r];
#pragma unroll
                for (int j = 0; j < DPT; ++j) O[r][j] *= al;
            }
        }
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            float v[DPT];
#pragma unroll
            for (int j = 0; j < DPT / 2; ++j) {
                v[2 * j] = __uint_as_float(vraw[kk][j] << 16);
                v[2 * j + 1] = __uint_as_float(vraw[kk][j] & 0xffff0000u);
            }
            float pr[QR];
#pragma unroll
            for (int r4 = 0; r4 < QR / 4; ++r4) {
                const float4 t = *reinterpret_cast<const float4*>(sPw + kk * 8 + r4 * 4);
                pr[r4 * 4] = t.x; pr[r4 * 4 + 1] = t.y; pr[r4 * 4 + 2] = t.z; pr[r4 * 4 + 3] = t.w;
            }
#pragma unroll
            for (int r = 0; r < QR; ++r)
#pragma unroll
                for (int j = 0; j < DPT; ++j) O[r][j] = fmaf(pr[r], v[j], O[r][j]);
        }
    }
    // row sums over the 8 lanes that share t4
#pragma unroll
    for (int o = 4; o <= 16; o <<= 1) {
        z0 += __shfl_xor_sync(0xffffffffu, z0, o);
        z1 += __shfl_xor_sync(0xffffffffu, z1, o);
    }
    if (g == 0) {
        sred[(warp * 8 + 2 * t4) * 2 + 0] = m0;
        sred[(warp * 8 + 2 * t4) * 2 + 1] = z0;
        sred[(warp * 8 + 2 * t4 + 1) * 2 + 0] = m1;
        sred[(warp * 8 + 2 * t4 + 1) * 2 + 1] = z1;
    }
#pragma unroll
    for (int r = 0; r < QR; ++r)
#pragma unroll
        for (int j = 0; j < DPT; ++j) sO[(warp * QR + r) * D + lane * DPT + j] = O[r][j];
    __syncthreads();
    if (tid < 8) {
        float m = SHOTKV_NEG_INF;
        for (int w = 0; w < 8; ++w) m = fmaxf(m, sred[(w * 8 + tid) * 2]);
        float z = 0.f;
        for (int w = 0; w < 8; ++w) z += sred[(w * 8 + tid) * 2 + 1] * ex2f(sred[(w * 8 + tid) * 2] - m);
        sfin[tid * 2] = m;
        sfin[tid * 2 + 1] = z > 0.f ? 1.f / z : 0.f;
    }
    __syncthreads();
    for (int idx = tid; idx < p.G * D; idx += 256) {
        const int r = idx / D, dim = idx - r * D;
        const float m = sfin[r * 2];
        float o = 0.f;
        for (int w = 0; w < 8; ++w) {
            const float mw = sred[(w * 8 + r) * 2];
            if (mw != SHOTKV_NEG_INF) o += sO[(w * QR + r) * D + dim] * ex2f(mw - m);
        }
        p.out[((size_t)bl * p.H + (size_t)hk * p.G + r) * D + dim] = o * sfin[r * 2 + 1];
    }
    for (int j = tid; j < n; j += 256) {
        float s = 0.f;
        for (int r = 0; r < p.G; ++r) s += ex2f(sdec[r * p.Dcap + j] - sfin[r * 2]) * sfin[r * 2 + 1];
        p.partial[(size_t)u * p.Dcap + j] = s;
    }
}

// acc[bl][j] += sum over kv heads of partial (fixed order); the new entry starts from 0.
__global__ void decode_accumulate_kernel(const float* __restrict__ partial, int Hkv, int Dcap, int n_old, int T_old,
                                         float* __restrict__ acc, int* __restrict__ born) {
    const int bl = blockIdx.x;
    for (int j = threadIdx.x; j <= n_old; j += blockDim.x) {
        float s = 0.f;
        for (int h = 0; h < Hkv; ++h) s += partial[((size_t)bl * Hkv + h) * Dcap + j];
        const float prev = j == n_old ? 0.f : acc[(size_t)bl * Dcap + j];
        acc[(size_t)bl * Dcap + j] = prev + s;
        if (j == n_old) born[(size_t)bl * Dcap + j] = T_old;
    }
}

// Top-k of the n decode entries of one (b, l) by (acc descending, index ascending); writes the
// kept positions in ascending order and compacts acc and born.  Shared: n floats + 3n ints + scan.
// Entries born at or after `protect_from` rank before all others (an option beyond the paper's
// rule; pass a value above every step number to protect nothing).
__global__ void __launch_bounds__(kSelectThreads) decode_rank_kernel(float* __restrict__ acc, int* __restrict__ born,
                                                                    int Dcap, int n, int k, int protect_from,
                                                                    int* __restrict__ keep_pos) {
    extern __shared__ __align__(16) unsigned char sm[];
    float* a = reinterpret_cast<float*>(sm);
    int* bs = reinterpret_cast<int*>(a + n);
    int* kf = bs + n;     // keep flag
    int* ds = kf + n;     // keep flag, then its exclusive scan = destination
    int* tmp = ds + n;
    const int bl = blockIdx.x, tid = threadIdx.x;
    for (int j = tid; j < n; j += kSelectThreads) {
        const float v = acc[(size_t)bl * Dcap + j];
        a[j] = v == v ? v : SHOTKV_NEG_INF;      // keep the order total even if a score is NaN
        bs[j] = born[(size_t)bl * Dcap + j];
    }
    __syncthreads();
    const float top = __int_as_float(0x7f800000);
    for (int j = tid; j < n; j += kSelectThreads) {
        const float v = bs[j] >= protect_from ? top : a[j];
        int rank = 0;
        for (int i = 0; i < n; ++i) {
            const float w = bs[i] >= protect_from ? top : a[i];
            rank += (w > v) || (w == v && i < j);
        }
        kf[j] = ds[j] = rank < k;
    }
    __syncthreads();
    block_exclusive_scan(ds, n, tmp);
    for (int j = tid; j < n; j += kSelectThreads) {
        if (kf[j]) {
            const int dst = ds[j];
            keep_pos[(size_t)bl * Dcap + dst] = j;
            acc[(size_t)bl * Dcap + dst] = a[j];
            born[(size_t)bl * Dcap + dst] = bs[j];
        }
    }
}

// In-place compaction of the decode K or V rows of one (b, l, kv head): row j <- row keep_pos[j].
// keep_pos is ascending with keep_pos[j] >= j, so a pass that first loads 256/VPR source rows and
// then, after a barrier, stores them at rows [c, c+256/VPR) never overwrites a later source.
template <int D>
__global__ void __launch_bounds__(256) decode_compact_kernel(__nv_bfloat16* Kd, __nv_bfloat16* Vd,
                                                            const int* __restrict__ keep_pos, int Hkv, int Dcap,
                                                            int k) {
    constexpr int VPR = D / 8;
    constexpr int ROWS = 256 / VPR;
    const int u = blockIdx.x;
    const int bl = u / Hkv;
    uint4* X = reinterpret_cast<uint4*>((blockIdx.y == 0 ? Kd : Vd) + (size_t)u * Dcap * D);
    const int* kp = keep_pos + (size_t)bl * Dcap;
    const int row_in = threadIdx.x / VPR, v = threadIdx.x % VPR;
    for (int c = 0; c < k; c += ROWS) {
        const int j = c + row_in;
        uint4 val = make_uint4(0, 0, 0, 0);
        const bool ok = j < k;
        if (ok) val = X[(size_t)kp[j] * VPR + v];
        __syncthreads();
        if (ok) X[(size_t)j * VPR + v] = val;
        __syncthreads();
    }
}

}  // namespace shotkv
