// Second pass of per-token importance on the 5th-generation tensor cores.
//
// With every window row's final maximum M_r and 1/Z_r known (row_stats_kernel), the logits are
// recomputed, normalised and summed over the rows: token_importance[t] = sum_r alpha[r][t].
// The product is taken transposed, S^T = K_tile . Q^T (A = a tile of 128 keys, B = all R window
// rows of the unit, N = 128 or 256 in one instruction), so that a key is a tensor-memory lane and
// the window rows run along the columns: the sum over rows is then a sum inside one thread, with
// no exchange between lanes.  Same persistent structure, work items, TMA producer and barrier
// protocol as the scoring kernels (score_tc.cuh); Q is laid out in shared memory k-block major so
// that the R rows of one 64-element k block are contiguous, as the B operand needs.
//
// Epilogue: eight warps in two groups; a warp owns 32 keys (its tensor-memory lanes), a group
// half of the window rows.  Per row the constants (-M_r, 1/Z_r) come from shared memory as
// broadcast reads.  The second group hands its partial sums to the first through a two-slot
// shared-memory ring guarded by mbarriers; the first adds them in a fixed order and stores.
#pragma once
#include "score_fast.cuh"

namespace shotkv {

struct ColsumTcParams {
    ScoreTcParams base;       // work partition (nchunk, chunk_keys, total_items, L, Hkv, N, W, R, Rpad, scale_log2, err)
    const float* row_m;       // [U][Rpad]
    const float* row_invz;    // [U][Rpad]
    float* imp;               // [U][N]
};

template <int D, int MB>
struct ColsumTcCfg {
    static constexpr int kSub = D / 64;
    static constexpr int kSubBytes = 128 * 128;
    static constexpr int kQBytes = MB * kSub * kSubBytes;
    static constexpr int kStageBytes = kSub * kSubBytes;
    static constexpr int kStages = D == 128 ? 4 : 6;              // even: see mma_role_transposed
    static constexpr int kBarBytes = 1024;
    static constexpr int kRows = 128 * MB;
    // per epilogue warp: the constants of its half of the rows, [rows/4] float4 (-M_r, -M_r+1, 1/Z_r, 1/Z_r+1)
    // and causal limits [rows/2] int; then the hand-over slots [4 quads][2][32] float
    static constexpr int kCombBytes = 8 * ((kRows / 4) * 16 + (kRows / 2) * 4) + 4 * 2 * 32 * 4;
    static constexpr int kSmemBytes = kQBytes + kStages * kStageBytes + kBarBytes + kCombBytes + 1024;
    static constexpr int kEpiWarps = 8;
    static constexpr int kThreads = 128 + kEpiWarps * 32;
};

namespace tc {

// One thread: S^T[128 keys x R rows] = K_tile . Q^T, accumulators double-buffered in tensor memory
// (buffer a at column a * 128 * MB).  Thread `which` of two issues the tiles of its parity.
template <int D, int MB, class Cfg>
__device__ __forceinline__ void mma_role_transposed(const Pipe<Cfg>& pp, const ScoreTcParams& p, int item_begin,
                                                    int item_end, int which) {
    constexpr int KSTEPS = D / 16, NST = Cfg::kStages, TN = kTileKeys, NR = 128 * MB;
    constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NR >> 3) << 17) | ((128u >> 4) << 24);
    // two threads on alternate tiles: only an even ring lets each meet every stage it uses on every turn
    static_assert(NST % 2 == 0, "each MMA thread must meet every stage it uses on every turn of the K ring");
    int stage = 0, acc = 0, cur_u = -1;
    uint32_t fphase = 0, qfphase = 0, tephase0 = 1, tephase1 = 1;
    bool ok = true;
    for (int it = item_begin; it < item_end && ok; ++it) {
        const int u = it / p.nchunk, j = it - u * p.nchunk;
        const int lo = j * p.chunk_keys, hi = min(p.N, lo + p.chunk_keys);
        const int nt = (hi - lo + TN - 1) / TN;
        if (nt <= 0) continue;
        if (u != cur_u) {
            if (cur_u >= 0) umma_commit(pp.qempty());
            if (!(ok = mbar_wait_relaxed(pp.qfull(), qfphase, pp.abort_flag, p.err, p.wait_cycles))) break;
            qfphase ^= 1;
            cur_u = u;
        }
        for (int t = 0; t < nt; ++t) {
            if (acc == which) {
                if (!(ok = mbar_wait_relaxed(pp.full(stage), fphase, pp.abort_flag, p.err, p.wait_cycles))) break;
                const uint32_t tph = acc ? tephase1 : tephase0;
                if (!(ok = mbar_wait_relaxed(pp.tempty(acc, 0), tph, pp.abort_flag, p.err, p.wait_cycles))) break;
                fence_after_sync();
                const uint32_t kb = pp.sK + stage * Cfg::kStageBytes;
                const uint32_t d_tmem = pp.tmem_base + (uint32_t)(acc * NR);
#pragma unroll
                for (int ks = 0; ks < KSTEPS; ++ks) {
                    const uint32_t a_addr = kb + (ks >> 2) * Cfg::kSubBytes + (ks & 3) * 32;
                    const uint32_t b_addr = pp.sQ + (ks >> 2) * (MB * Cfg::kSubBytes) + (ks & 3) * 32;
                    umma_bf16(d_tmem, smem_desc(a_addr), smem_desc(b_addr), idesc, ks > 0);
                }
                umma_commit(pp.tfull(acc, 0));
                if (acc) tephase1 ^= 1; else tephase0 ^= 1;
                umma_commit(pp.empty(stage));
            }
            if (++stage == NST) {
                stage = 0;
                fphase ^= 1;
            }
            acc ^= 1;
        }
    }
}

}  // namespace tc

template <int D, int MB, int PE>
__global__ void __launch_bounds__(ColsumTcCfg<D, MB>::kThreads, 1)
    colsum_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const int q_box_rows,
                     const int k_box_rows, const ColsumTcParams cp) {
    using Cfg = ColsumTcCfg<D, MB>;
    constexpr int TN = tc::kTileKeys, ROWS = Cfg::kRows, RG = ROWS / 2, NCH = RG / 32;
    const ScoreTcParams& p = cp.base;
    extern __shared__ unsigned char smem_raw[];
    tc::Pipe<Cfg> pp;
    tc::pipe_setup(pp, smem_raw, Cfg::kEpiWarps, 4 * 2 * 2, 2);     // extra barriers: [quad][slot][full, empty]
    float4* cst = reinterpret_cast<float4*>(tc::pipe_scratch(pp, smem_raw));    // [8 warps][RG / 2]
    int* plim_s = reinterpret_cast<int*>(cst + 8 * (RG / 2));                      // [8 warps][RG]
    float* slots = reinterpret_cast<float*>(plim_s + 8 * RG);                      // [4][2][32]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long total = p.total_items;
    const int item_begin = (int)(total * blockIdx.x / gridDim.x);
    const int item_end = (int)(total * (blockIdx.x + 1) / gridDim.x);

    // Every window row is a column of the accumulator and all columns are summed by one thread, so
    // the rows of the Q area that no copy ever writes (fewer than 128 query rows in all) must hold
    // numbers: zero the area once, and make that visible to the tensor core's reads.
    {
        unsigned char* q_area = smem_raw + (pp.sQ - smem_u32(smem_raw));
        for (int i = threadIdx.x * 16; i < Cfg::kQBytes; i += blockDim.x * 16) *reinterpret_cast<uint4*>(q_area + i) = make_uint4(0, 0, 0, 0);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
    }

    if (warp == 0) {
        if (lane == 0) tc::producer_role<D, MB, false, true>(pp, &tmQ, &tmK, q_box_rows, k_box_rows, p, item_begin, item_end);
    } else if (warp == 1 || warp == 2) {
        if (lane == 0) tc::mma_role_transposed<D, MB>(pp, p, item_begin, item_end, warp - 1);
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ epilogue
        const int e = warp - 4, g = e >> 2, quad = warp & 3;
        const int r0 = g * RG;                             // first window row (accumulator column) of this group
        const float scale = p.scale_log2;
        const uint64_t sc2 = tc::pack2(scale, scale);
        const float c1 = scale * (1.f / 254.f);
        float4* cu = cst + e * (RG / 2);                   // this warp's own copy of its rows' constants
        int* pl = plim_s + e * RG;
        int acc = 0, cur_u = -1, ntile = 0;
        uint32_t tfphase0 = 0, tfphase1 = 0;
        bool ok = true;
        for (int it = item_begin; it < item_end && ok; ++it) {
            const int u = it / p.nchunk, j = it - u * p.nchunk;
            const int lo = j * p.chunk_keys, hi = min(p.N, lo + p.chunk_keys);
            const int nt = (hi - lo + TN - 1) / TN;
            if (nt <= 0) continue;
            if (u != cur_u) {
                cur_u = u;
                __syncwarp();                              // the previous unit's constants have been read
                for (int rr = lane; rr < RG; rr += 32) {
                    const int r = r0 + rr;
                    const bool live = r < p.R;
                    const float m = live ? cp.row_m[(size_t)u * p.Rpad + r] : 0.f;
                    const float iz = live ? cp.row_invz[(size_t)u * p.Rpad + r] : 0.f;
                    float* c4 = reinterpret_cast<float*>(cu + (rr >> 1));
                    // first two components: the additive constant of the row's exponential, -M_r where the
                    // column pair goes to the special-function unit, (126 - M_r) / 254 where it goes to the
                    // FMA pipe (see exp2_fma2); a row without weight gets 1/Z = 0 and a constant that exponentiates to
                    // (nearly) zero, so that no infinity meets that zero
                    const bool has = live && iz > 0.f;
                    c4[rr & 1] = tc::pair_on_fma<PE>((rr >> 1) & 15) ? (has ? (126.f - m) * (1.f / 254.f) : -4.f)
                                                                     : (has ? -m : SHOTKV_NEG_INF);
                    c4[2 + (rr & 1)] = has ? iz : 0.f;
                    pl[rr] = live ? p.N - p.W + (r % p.W) : -1;
                }
                __syncwarp();
            }
            for (int t = 0; t < nt; ++t) {
                const uint32_t tph = acc ? tfphase1 : tfphase0;
                if (!__all_sync(0xffffffffu, tc::mbar_try(pp.tfull(acc, 0), tph))) {
                    bool w = lane == 0 ? tc::mbar_wait(pp.tfull(acc, 0), tph, pp.abort_flag, p.err, p.wait_cycles) : true;
                    w = __shfl_sync(0xffffffffu, w, 0);
                    if (!w) ok = false;
                }
                if (!ok) break;
                if (acc) tfphase1 ^= 1; else tfphase0 ^= 1;
                tc::fence_after_sync();
                const int key = lo + t * TN + quad * 32 + lane;
                const uint32_t taddr = pp.tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * ROWS + r0);
                const bool plain = lo + t * TN + TN <= p.N - p.W + 1;       // every key of the tile counts for every row
                uint64_t s2[2] = {0ull, 0ull};
                uint32_t r[32];
#pragma unroll 1
                for (int c = 0; c < NCH; ++c) {
                    tc::tmem_ld32_sync(r, taddr + c * 32);
                    if (c == NCH - 1) {
                        tc::fence_before_sync();
                        __syncwarp();
                        if (lane == 0) tc::mbar_arrive(pp.tempty(acc, 0));
                    }
                    // alpha of the pair of rows (2 jp, 2 jp + 1) at this thread's key, times 1/Z, added to the sums
                    auto pair_term = [&](int jp, bool masked) {
                        const float4 k4 = cu[c * 16 + jp];
                        uint64_t e2;
                        if (tc::pair_on_fma<PE>(jp)) {
                            e2 = tc::exp2_from_unit2(tc::fma_sat(SKV_F(r, 2 * jp), c1, k4.x), tc::fma_sat(SKV_F(r, 2 * jp + 1), c1, k4.y));
                        } else {
                            const uint64_t x2 = tc::ffma2(tc::pack2(SKV_F(r, 2 * jp), SKV_F(r, 2 * jp + 1)), sc2, tc::pack2(k4.x, k4.y));
                            float xa, xb;
                            tc::unpack2(x2, xa, xb);
                            e2 = tc::pack2(ex2f(xa), ex2f(xb));
                        }
                        if (masked) {                                       // after a row's own position: no weight
                            float ea, eb;
                            tc::unpack2(e2, ea, eb);
                            e2 = tc::pack2(key > pl[c * 32 + 2 * jp] ? 0.f : ea, key > pl[c * 32 + 2 * jp + 1] ? 0.f : eb);
                        }
                        s2[jp & 1] = tc::ffma2(e2, tc::pack2(k4.z, k4.w), s2[jp & 1]);
                    };
                    if (plain) {
#pragma unroll
                        for (int jp = 0; jp < 16; ++jp) pair_term(jp, false);
                    } else {
#pragma unroll
                        for (int jp = 0; jp < 16; ++jp) pair_term(jp, true);
                    }
                }
                float sum;
                {
                    float a0, a1, a2, a3;
                    tc::unpack2(s2[0], a0, a1);
                    tc::unpack2(s2[1], a2, a3);
                    sum = (a0 + a1) + (a2 + a3);
                }
                // hand-over: group 1 posts, group 0 adds and stores
                const int slot = ntile & 1;
                const uint32_t par = (uint32_t)(ntile >> 1) & 1u;
                const int bs = (quad * 2 + slot) * 2;                       // barrier pair of (quad, slot)
                float* sl = slots + (quad * 2 + slot) * 32;
                if (g == 1) {
                    if (ntile >= 2) {
                        bool w = lane == 0 ? tc::mbar_wait(pp.extra_bar(bs + 1), par ^ 1u, pp.abort_flag, p.err, p.wait_cycles) : true;
                        w = __shfl_sync(0xffffffffu, w, 0);
                        __syncwarp();
                        if (!w) ok = false;
                    }
                    sl[lane] = sum;
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(pp.extra_bar(bs));
                } else {
                    bool w = lane == 0 ? tc::mbar_wait(pp.extra_bar(bs), par, pp.abort_flag, p.err, p.wait_cycles) : true;
                    w = __shfl_sync(0xffffffffu, w, 0);
                    __syncwarp();
                    if (!w) ok = false;
                    sum += sl[lane];
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(pp.extra_bar(bs + 1));
                    if (key < hi) cp.imp[(size_t)u * p.N + key] = sum;
                }
                ++ntile;
                acc ^= 1;
            }
        }
    }

    tc::fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tc::fence_after_sync();
        tc::tmem_dealloc(pp.tmem_base, 512);
    }
}

}  // namespace shotkv
