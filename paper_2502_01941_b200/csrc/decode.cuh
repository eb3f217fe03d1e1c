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

// ---- helpers of the fused step ---------------------------------------------------------------
// 16 bytes global -> shared without a register stage; `bytes` = 16 copies, 0 writes zeros.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// Four 8x8 bf16 matrices from shared memory, transposed: register i of lane (g, t4) holds
// elements [2*t4][g] and [2*t4 + 1][g] of the matrix whose row addresses lanes 8i..8i+7 supplied.
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// Two floats as a bf16 pair (round to nearest even), low half = a.
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// Shared-memory staging of the fused step: every warp owns a ring of kStages stages, a stage
// holding the 16 key rows and the 16 value rows of one block, unpadded, with the 16-byte chunks of a
// row permuted so that the reads are free of bank conflicts: keys (read back as 16 bytes per lane,
// two rows per quarter-warp) with chunk ^ 4*(row & 1), values (read by ldmatrix, eight rows per
// matrix) with chunk ^ (row & 7).
template <int D>
struct AttendCfg {
    static constexpr int kWarps = 4;                              // warps per CTA
    static constexpr int kStages = 2;                             // blocks in the ring: one in use, one in flight (three CTAs fit an SM)
    static constexpr int kRowBytes = D * 2;
    static constexpr int kTileBytes = 16 * kRowBytes;             // 16 rows of keys (or of values)
    static constexpr int kStageBytes = 2 * kTileBytes;
    static constexpr int kRingBytes = kWarps * kStages * kStageBytes;
    static constexpr int kOBytes = kWarps * 8 * D * 4;            // the warps' outputs for the final merge (reuses the ring)
    static_assert(kOBytes <= kRingBytes, "the merge area must fit into the ring");
};

// The same step with the attention output fused in: o_h = sum_t alpha_{t,h} v_t over the kept
// prefill entries and the decode entries, with the very weights the decoding score sums, so that
// scoring adds no pass over K to a decode step that has to read K and V anyway.
//
// HBM-bound, and what it takes to stay there is bytes in flight: a warp that loads a block's keys
// into registers and then waits for them is idle for the whole (loaded) memory latency, and the
// accumulators of the output leave too few registers for enough such warps.  So nothing is loaded
// into registers from global memory here: key and value rows go global -> shared by cp.async one
// block ahead of their use, into a per-warp ring (measured: two stages with three CTAs on an SM beat three stages with two).
//
// Both products run on the tensor cores, transposed so that the few query rows of a group are the
// narrow N = 8 side.  Per block of 16 keys a warp computes S^T[rows x keys] = Q . K^T with the
// group's query rows as the A operand (held in registers) and the key rows as B fragments (16
// contiguous bytes per lane and 32-dim block; the same k-index permutation on both operands).
// The accumulator fragment of that product -- lane (g, t4) holds row g, keys 2*t4, 2*t4+1,
// 8+2*t4, 9+2*t4 -- is, after the exponential, exactly the B fragment of O^T[dims x rows] =
// V^T . P^T, so the weights never leave their registers; they enter as a bf16 pair (high part plus
// remainder: relative error 2^-17) in two MMAs per 16 dimensions, and ldmatrix.trans turns the
// value rows into the A fragments of V^T.  Online softmax per warp with a running maximum per
// query row (lanes that share g); the warps' (m, z, O) are merged at the end in warp order.
template <int D>
__global__ void __launch_bounds__(AttendCfg<D>::kWarps * 32, 3) decode_attend_kernel(const DecodeParams p) {
    using Cfg = AttendCfg<D>;
    constexpr int NB = D / 32;     // 32-dim blocks
    constexpr int VPR = D / 8;     // 16-byte chunks per row
    constexpr int MT = D / 16;     // 16-dim tiles of the output
    constexpr int NW = Cfg::kWarps, NS = Cfg::kStages, NT = NW * 32;
    extern __shared__ __align__(16) unsigned char dsm[];
    float* sdec = reinterpret_cast<float*>(dsm);             // [8][Dcap]
    float* sred = sdec + 8 * p.Dcap;                         // [NW warps][8 rows][2]
    float* sfin = sred + NW * 8 * 2;                         // [8 rows][2]  (m, 1/Z)
    unsigned char* ring = reinterpret_cast<unsigned char*>(sfin + 16);   // [NW][NS][keys | values][16 rows][D bf16]; later [NW][8 rows][D] floats
    float* sO = reinterpret_cast<float*>(ring);

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
    const uint4* Vc_u = reinterpret_cast<const uint4*>(p.Vc + (size_t)u * p.Mcap * D);

    // append the new token's key and value as decode entry n_old
    if (tid < VPR) Kd_u[(size_t)p.n_old * VPR + tid] = knew_u[tid];
    else if (tid < 2 * VPR) Vd_u[(size_t)p.n_old * VPR + (tid - VPR)] = vnew_u[tid - VPR];

    // query row g of the group as A fragments (rows 8..15 of the 16-row operand are zero)
    uint4 qf[NB];
    {
        const uint4* qrow = reinterpret_cast<const uint4*>(p.q + ((size_t)bl * p.H + (size_t)hk * p.G + g) * D);
#pragma unroll
        for (int kb = 0; kb < NB; ++kb) qf[kb] = g < p.G ? qrow[kb * 4 + t4] : make_uint4(0, 0, 0, 0);
    }

    // this warp's ring.  A lane copies chunk (lane % VPR) of rows lane / VPR + k * (32 / VPR); rows
    // past the end are filled with zeros (a weight of zero must not meet a stray NaN).
    const uint32_t wring = smem_u32(ring) + (uint32_t)(warp * NS * Cfg::kStageBytes);
    auto fetch_block = [&](int base, int stage) {
        constexpr int RPI = 32 / VPR;                       // rows per warp-wide copy
        const int c = lane % VPR;
        const uint32_t st = wring + (uint32_t)(stage * Cfg::kStageBytes);
#pragma unroll
        for (int k = 0; k < 16 / RPI; ++k) {
            const int rr = lane / VPR + k * RPI;
            const int i = base + rr;
            const bool valid = i < Ktot;
            const bool fresh = i - M == p.n_old;            // the token appended by this very step
            const uint4* ksrc = i < M ? Kc_u + (size_t)i * VPR : (fresh ? knew_u : Kd_u + (size_t)(i - M) * VPR);
            const uint4* vsrc = i < M ? Vc_u + (size_t)i * VPR : (fresh ? vnew_u : Vd_u + (size_t)(i - M) * VPR);
            cp_async16(st + (uint32_t)(rr * Cfg::kRowBytes + ((c ^ ((rr & 1) << 2)) << 4)), valid ? ksrc + c : knew_u, valid ? 16 : 0);
            cp_async16(st + (uint32_t)(Cfg::kTileBytes + rr * Cfg::kRowBytes + ((c ^ (rr & 7)) << 4)), valid ? vsrc + c : vnew_u, valid ? 16 : 0);
        }
        cp_async_commit();
    };
    // ldmatrix row of this lane: matrix lane/8 = (keys 0-7 | 8-15) x (dims +0 | +8), row lane%8
    const int ldm_row = ((lane >> 4) & 1) * 8 + (lane & 7), ldm_hi = (lane >> 3) & 1;

    float O[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int q = 0; q < 4; ++q) O[mt][q] = 0.f;
    // running maximum of query row g over this warp's keys (the same in the 4 lanes that share g);
    // z: this lane's part of the row sum relative to it
    float m = SHOTKV_NEG_INF, z = 0.f;
    // blocks are requested NS - 1 ahead; one copy group per block, empty past the end, so that
    // "at most NS - 1 groups pending" always means this block's rows have landed
    constexpr int STRIDE = NW * 16;
    int stage = 0;
#pragma unroll
    for (int k = 0; k < NS - 1; ++k) {
        if (warp * 16 + k * STRIDE < Ktot) fetch_block(warp * 16 + k * STRIDE, k);
        else cp_async_commit();
    }
    for (int base = warp * 16; base < Ktot; base += STRIDE) {
        __syncwarp();                                       // every lane has read the stage the next copy overwrites
        {
            const int nb = base + (NS - 1) * STRIDE;
            if (nb < Ktot) fetch_block(nb, stage == 0 ? NS - 1 : stage - 1);
            else cp_async_commit();
        }
        cp_async_wait<NS - 1>();                            // this block's rows have landed (later blocks' may be in flight)
        __syncwarp();
        const uint32_t st = wring + (uint32_t)(stage * Cfg::kStageBytes);
        // keys base+g and base+8+g as B fragments
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};   // keys base+0..7 and base+8..15
#pragma unroll
        for (int kb = 0; kb < NB; ++kb) {
            const uint32_t off = (uint32_t)(((kb * 4 + t4) ^ ((g & 1) << 2)) << 4);
            uint4 ka, kb8;
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(ka.x), "=r"(ka.y), "=r"(ka.z), "=r"(ka.w) : "r"(st + (uint32_t)(g * Cfg::kRowBytes) + off));
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(kb8.x), "=r"(kb8.y), "=r"(kb8.z), "=r"(kb8.w) : "r"(st + (uint32_t)((g + 8) * Cfg::kRowBytes) + off));
            const uint32_t a0[4] = {qf[kb].x, 0u, qf[kb].y, 0u};
            const uint32_t a1[4] = {qf[kb].z, 0u, qf[kb].w, 0u};
            mma_bf16_16816(s0, a0, ka.x, ka.y);
            mma_bf16_16816(s0, a1, ka.z, ka.w);
            mma_bf16_16816(s1, a0, kb8.x, kb8.y);
            mma_bf16_16816(s1, a1, kb8.z, kb8.w);
        }
        // this lane: row g, keys base + {2*t4, 2*t4+1, 8+2*t4, 9+2*t4}
        const int k0 = base + 2 * t4;
        float x[4];
        x[0] = k0 < Ktot ? s0[0] * p.scale_log2 : SHOTKV_NEG_INF;
        x[1] = k0 + 1 < Ktot ? s0[1] * p.scale_log2 : SHOTKV_NEG_INF;
        x[2] = k0 + 8 < Ktot ? s1[0] * p.scale_log2 : SHOTKV_NEG_INF;
        x[3] = k0 + 9 < Ktot ? s1[1] * p.scale_log2 : SHOTKV_NEG_INF;
        if (g < p.G) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int key = k0 + (q & 1) + (q >> 1) * 8;
                if (key >= M && key < Ktot) sdec[g * p.Dcap + (key - M)] = x[q];
            }
        }
        float bm = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
        bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 1));
        bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 2));
        const float mn = fmaxf(m, bm);
        const float mu = mn == SHOTKV_NEG_INF ? 0.f : mn;
        const float al = ex2f(m - mu);                      // rescale of what was summed so far
        float pw[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) pw[q] = ex2f(x[q] - mu);
        z = z * al + (pw[0] + pw[1]) + (pw[2] + pw[3]);
        const bool changed = __any_sync(0xffffffffu, mn != m);
        m = mn;
        if (changed) {
            // the output fragments hold rows 2*t4 and 2*t4+1: their factors live in lanes 8*t4 and 8*t4+4
            const float f0 = __shfl_sync(0xffffffffu, al, 8 * t4), f1 = __shfl_sync(0xffffffffu, al, 8 * t4 + 4);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                O[mt][0] *= f0; O[mt][1] *= f1; O[mt][2] *= f0; O[mt][3] *= f1;
            }
        }
        // weights as B fragments of the second product: high bf16 part and remainder
        const uint32_t h0 = pack_bf16(pw[0], pw[1]), h1 = pack_bf16(pw[2], pw[3]);
        const uint32_t l0 = pack_bf16(pw[0] - __uint_as_float(h0 << 16), pw[1] - __uint_as_float(h0 & 0xffff0000u));
        const uint32_t l1 = pack_bf16(pw[2] - __uint_as_float(h1 << 16), pw[3] - __uint_as_float(h1 & 0xffff0000u));
        const uint32_t vrow = st + (uint32_t)(Cfg::kTileBytes + ldm_row * Cfg::kRowBytes);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            uint32_t a[4];
            ldmatrix_x4_trans(a, vrow + (uint32_t)((((2 * mt + ldm_hi) ^ (ldm_row & 7))) << 4));
            mma_bf16_16816(O[mt], a, h0, h1);
            mma_bf16_16816(O[mt], a, l0, l1);
        }
        stage = stage + 1 == NS ? 0 : stage + 1;
    }
    cp_async_wait<0>();
    // row sums over the 4 lanes that share g
    z += __shfl_xor_sync(0xffffffffu, z, 1);
    z += __shfl_xor_sync(0xffffffffu, z, 2);
    if (t4 == 0) {
        sred[(warp * 8 + g) * 2 + 0] = m;
        sred[(warp * 8 + g) * 2 + 1] = z;
    }
    __syncthreads();                                        // all warps are done with their rings
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        sO[(warp * 8 + 2 * t4) * D + mt * 16 + g] = O[mt][0];
        sO[(warp * 8 + 2 * t4 + 1) * D + mt * 16 + g] = O[mt][1];
        sO[(warp * 8 + 2 * t4) * D + mt * 16 + 8 + g] = O[mt][2];
        sO[(warp * 8 + 2 * t4 + 1) * D + mt * 16 + 8 + g] = O[mt][3];
    }
    if (tid < 8) {
        float mm = SHOTKV_NEG_INF;
        for (int w = 0; w < NW; ++w) mm = fmaxf(mm, sred[(w * 8 + tid) * 2]);
        float zz = 0.f;
        for (int w = 0; w < NW; ++w) zz += sred[(w * 8 + tid) * 2 + 1] * ex2f(sred[(w * 8 + tid) * 2] - mm);
        sfin[tid * 2] = mm;
        sfin[tid * 2 + 1] = zz > 0.f ? 1.f / zz : 0.f;
    }
    __syncthreads();
    for (int idx = tid; idx < p.G * D; idx += NT) {
        const int r = idx / D, dim = idx - r * D;
        const float mm = sfin[r * 2];
        float o = 0.f;
        for (int w = 0; w < NW; ++w) {
            const float mw = sred[(w * 8 + r) * 2];
            if (mw != SHOTKV_NEG_INF) o += sO[(w * 8 + r) * D + dim] * ex2f(mw - mm);
        }
        p.out[((size_t)bl * p.H + (size_t)hk * p.G + r) * D + dim] = o * sfin[r * 2 + 1];
    }
    for (int j = tid; j < n; j += NT) {
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
