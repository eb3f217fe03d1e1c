// Window attention scoring for units of 128 window rows or fewer (one 128-row block of Q), the
// kernel the prefill path runs first on them: the same TMA producer, MMA issuers, work items and
// per-(piece, window row) outputs (m, z) as score_tc.cuh, with an epilogue arranged for
// throughput.  (Units of more than 128 rows go to score_stream.cuh, which shares the exponential
// helpers defined here.)
//
//   * Eight epilogue warps in two groups that split a tile's columns in halves; a thread is one
//     window row and one half.  When a piece is complete the second group hands its (m, z) to the
//     first through a small ring of shared-memory slots guarded by mbarriers, so no warp waits
//     for another at a piece end unless it is a whole ring ahead of it.  The code of the inner
//     loop is kept small and free of branches (one copy of the chunk arithmetic, one of the
//     boundary handling): the warps of three roles share the instruction cache.  Where pieces end
//     inside a chunk its exponentials are split between them by 0/1 masks from shared memory.
//   * No running maximum.  The reference exponent m of a (row, column half, work item) is fixed
//     from the item's first tile: that tile's row maximum lands on 2^-32, and every later logit
//     of the item is exponentiated against the same m.  fp32 leaves about 2^+158 above that point
//     and 2^-94 below it; what underflows is below 2^-94 of a term the row's own softmax
//     denominator contains, so it cannot matter to any score.  What overflows is caught: a
//     partial sum that is not below 1e30 marks its item in `redo`, and a second launch (the exact
//     kernel of score_tc.cuh with the same flags) recomputes marked items with a true running
//     maximum.
//   * One ex2 per logit is the ceiling of the special-function unit (16 lanes per clock per SM),
//     so PE of every 16 column pairs take their exponentials on the FMA pipe instead: round to nearest
//     integer n by the magic-number addition, a cubic in the remainder f in [-1/2, 1/2]
//     (relative error below 7.5e-5), and n added into the exponent field.  A saturating
//     multiply-add clamps the argument to [-126, 128] first, so the result is a normal number,
//     or +inf at the top.
#pragma once
#include "score_tc.cuh"

namespace shotkv {

template <int D>
struct ScoreFastCfg {
    static constexpr int kSub = D / 64;
    static constexpr int kSubBytes = 128 * 128;
    static constexpr int kQBytes = kSub * kSubBytes;
    static constexpr int kStageBytes = kSub * kSubBytes;
    // An even number: the two MMA threads take alternate tiles, so with an even ring each of them meets
    // a given stage every time round and its parity wait can never be a whole turn behind the barrier.
    // (Four 32 KB stages measure the same as five.)
    static constexpr int kStages = D == 128 ? 4 : 6;
    static constexpr int kBarBytes = 2048;
    static constexpr int kRingDepth = 4;                       // hand-over slots between a row's column slices
    static constexpr int kRings = 4;                           // one per warp quarter
    static constexpr int kCombBytes = kRings * kRingDepth * 32 * 2 * 4;   // [ring][slot][lane][m, z]
    static constexpr int kSmemBytes = kQBytes + kStages * kStageBytes + kBarBytes + kCombBytes + 33 * 16 * 16 + 1024;   // + split masks
    static constexpr int kSlices = 2;                          // column slices of a tile
    static constexpr int kEpiWarps = 8;
    static constexpr int kThreads = 128 + kEpiWarps * 32;      // producer, two MMA issuers, one idle warp; epilogue
};

namespace tc {

constexpr float kRefShift = 32.f;        // the first tile's row maximum is exponentiated to 2^-32
constexpr float kRedoAbove = 1e30f;      // a partial sum at or above this sends its item to the exact kernel

// 2^x on the FMA pipe for two logits at a time, x = s * scale + neg.  One saturating
// multiply-add per logit maps x from [-126, 128] onto y in [0, 1] and so does the scaling, the
// shift and both clamps at once (c1 = scale / 254, c0 = (neg + 126) / 254; the grid of y costs
// x an absolute error below 8e-6).  Then, on packed pairs: t = 254 y + (1.5 * 2^23 - 126) rounds
// to the nearest integer n = round(x) in its low mantissa bits, t - (1.5 * 2^23 - 126) = n + 126
// exactly, g = (n + 126) - 254 y = -(x - n) lies in [-1/2, 1/2], a cubic in g gives 2^(x - n)
// (relative error below 7.5e-5) and n is added into the exponent field.  x >= 128 yields +inf,
// x <= -126 a number below 2^-125; nothing in between leaves the normal range.
__device__ __forceinline__ float fma_sat(float a, float b, float c) {
    float d;
    asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// 2^x for two values given as y = (x + 126) / 254 in [0, 1]
__device__ __forceinline__ uint64_t exp2_from_unit2(float ya, float yb) {
    constexpr float kMagic = 12582912.f - 126.f;
    const uint64_t y = pack2(ya, yb);
    const uint64_t t = ffma2(y, pack2(254.f, 254.f), pack2(kMagic, kMagic));
    const uint64_t fl = fadd2(t, pack2(-kMagic, -kMagic));
    const uint64_t g = ffma2(y, pack2(-254.f, -254.f), fl);
    uint64_t q = ffma2(pack2(-5.5171668e-02f, -5.5171668e-02f), g, pack2(2.4261112e-01f, 2.4261112e-01f));
    q = ffma2(q, g, pack2(-6.9326099e-01f, -6.9326099e-01f));
    q = ffma2(q, g, pack2(9.9992807e-01f, 9.9992807e-01f));
    float qa, qb, ta, tb;
    unpack2(q, qa, qb);
    unpack2(t, ta, tb);
    return pack2(__uint_as_float(__float_as_uint(qa) + (__float_as_uint(ta) << 23)),
                 __uint_as_float(__float_as_uint(qb) + (__float_as_uint(tb) << 23)));
}
__device__ __forceinline__ uint64_t exp2_fma2(float sa, float sb, float c1, float c0) {
    return exp2_from_unit2(fma_sat(sa, c1, c0), fma_sat(sb, c1, c0));
}

// Is column pair j (of 16) of a 32-column chunk exponentiated on the FMA pipe?  NP pairs are, spread evenly.
template <int NP>
__device__ __forceinline__ constexpr bool pair_on_fma(int j) {
    return NP > 0 && ((j + 1) * NP) / 16 != (j * NP) / 16;
}

// 2^(r[i] * scale + neg) for the column pair (2j, 2j+1), packed
template <int NP>
__device__ __forceinline__ uint64_t exp_pair(const uint32_t (&r)[32], int j, uint64_t sc2, uint64_t ng2, float c1, float c0) {
    if (pair_on_fma<NP>(j)) return exp2_fma2(SKV_F(r, 2 * j), SKV_F(r, 2 * j + 1), c1, c0);
    const uint64_t x2 = ffma2(pack2(SKV_F(r, 2 * j), SKV_F(r, 2 * j + 1)), sc2, ng2);
    float xa, xb;
    unpack2(x2, xa, xb);
    return pack2(ex2f(xa), ex2f(xb));
}

// z[0..1] (packed pairs: four running sums) += 2^(r[i] * scale + neg) over the 32 columns
template <int NP>
__device__ __forceinline__ void expacc32(const uint32_t (&r)[32], float scale, float neg, uint64_t (&z)[2]) {
    const uint64_t sc2 = pack2(scale, scale), ng2 = pack2(neg, neg);
    const float c1 = scale * (1.f / 254.f), c0 = (neg + 126.f) * (1.f / 254.f);
#pragma unroll
    for (int j = 0; j < 16; ++j) z[j & 1] = fadd2(z[j & 1], exp_pair<NP>(r, j, sc2, ng2, c1, c0));
}

// r[i] = 2^(r[i] * scale + neg) in place, the same split between the two pipes
template <int NP>
__device__ __forceinline__ void exp32_mixed(uint32_t (&r)[32], float scale, float neg) {
    const uint64_t sc2 = pack2(scale, scale), ng2 = pack2(neg, neg);
    const float c1 = scale * (1.f / 254.f), c0 = (neg + 126.f) * (1.f / 254.f);
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        float ea, eb;
        unpack2(exp_pair<NP>(r, j, sc2, ng2, c1, c0), ea, eb);
        r[2 * j] = __float_as_uint(ea);
        r[2 * j + 1] = __float_as_uint(eb);
    }
}

// ---- splitting a chunk's exponentials between the pieces that end inside it --------------------
// Table of 0/1 masks in shared memory: entry (nb, j) = {col 2j < nb, col 2j+1 < nb, col 2j >= nb,
// col 2j+1 >= nb} as 1.0 / 0.0, nb = 0..32 columns of the chunk that belong to the piece that ends.
constexpr int kSplitMaskBytes = 33 * 16 * 16;
__device__ __forceinline__ void build_split_masks(float4* mtab) {
    for (int i = threadIdx.x; i < 33 * 16; i += blockDim.x) {
        const int nb = i >> 4, j = i & 15;
        const float a = 2 * j < nb ? 1.f : 0.f, b = 2 * j + 1 < nb ? 1.f : 0.f;
        mtab[i] = make_float4(a, b, 1.f - a, 1.f - b);
    }
}
// 32 columns starting at key kc, all of which count for this thread's row, with one or more piece
// ends strictly inside (`pend` = end of the current piece; `flush` completes it and advances
// `pend`).  The pieces are peeled off in order: the columns before a piece's end go to its sum
// through a 0/1 mask (one packed multiply-add per column pair) and the complementary mask clears
// them from the chunk before the next piece is looked at; what is left starts the next piece.
// Half the instructions of a predicated addition per column, and no branch depends on a column.
template <int PE, class Flush>
__device__ __forceinline__ void peel_chunk(uint32_t (&r)[32], float scale, float neg, const float4* mtab, int kc,
                                           const int& pend, uint64_t (&z)[2], Flush&& flush) {
    exp32_mixed<PE>(r, scale, neg);
    while (pend < kc + 32) {
        const float4* mk = mtab + (pend - kc) * 16;
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            const float4 m4 = mk[q];
            const uint64_t e2 = pack2(SKV_F(r, 2 * q), SKV_F(r, 2 * q + 1));
            z[q & 1] = ffma2(e2, pack2(m4.x, m4.y), z[q & 1]);
            float ea, eb;
            unpack2(ffma2(e2, pack2(m4.z, m4.w), 0ull), ea, eb);
            r[2 * q] = __float_as_uint(ea);
            r[2 * q + 1] = __float_as_uint(eb);
        }
        flush();
    }
#pragma unroll
    for (int q = 0; q < 16; ++q) z[q & 1] = fadd2(z[q & 1], pack2(SKV_F(r, 2 * q), SKV_F(r, 2 * q + 1)));
}

}  // namespace tc

template <int D, int PE>
__global__ void __launch_bounds__(ScoreFastCfg<D>::kThreads, 1)
    score_fast_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const int q_box_rows,
                      const int k_box_rows, const ScoreTcParams p) {
    using Cfg = ScoreFastCfg<D>;
    constexpr int TN = tc::kTileKeys, MB = 1;
    constexpr int NSL = Cfg::kSlices, SLW = TN / NSL, NCH = SLW / 32, RD = Cfg::kRingDepth;
    extern __shared__ unsigned char smem_raw[];
    tc::stamp(p.clk, 0);
    tc::Pipe<Cfg> pp;
    tc::pipe_setup(pp, smem_raw, Cfg::kEpiWarps, Cfg::kRings * Cfg::kRingDepth * 2, 2);
    float* comb = tc::pipe_scratch(pp, smem_raw);     // [ring][slot][lane][m, z]
    float4* mtab = reinterpret_cast<float4*>(reinterpret_cast<unsigned char*>(comb) + Cfg::kCombBytes);   // split masks
    tc::build_split_masks(mtab);
    __syncthreads();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long total = p.total_items;
    const int item_begin = (int)(total * blockIdx.x / gridDim.x);
    const int item_end = (int)(total * (blockIdx.x + 1) / gridDim.x);

    if (warp == 0) {
        if (lane == 0) tc::producer_role<D, MB, false, false>(pp, &tmQ, &tmK, q_box_rows, k_box_rows, p, item_begin, item_end);
    } else if (warp == 1 || warp == 2) {
        if (lane == 0) tc::mma_role<D, MB, false, 2>(pp, p, item_begin, item_end, warp - 1);
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ epilogue
        // a warp may touch the 32 tensor-memory lanes given by its index modulo 4; any four
        // consecutive warps cover all 128 rows of a block
        const int slice = (warp - 4) >> 2, quad = warp & 3;   // column slice of every tile, lane quarter
        constexpr int blk = 0;                             // the one 128-row block of Q
        const int lrow = quad * 32 + lane;
        const int row = blk * 128 + lrow;
        const bool live = row < p.R;                       // padding rows: their Q was never loaded
        const int plim = live ? p.N - p.W + (row % p.W) : p.N - 1;
        const float scale = p.scale_log2;
        const int units_per_prompt = p.L * p.Hkv;
        int acc = 0, nflush = 0;
        uint32_t tfphase0 = 0, tfphase1 = 0;
        bool ok = true;
        for (int it = item_begin; it < item_end && ok; ++it) {
            const int u = it / p.nchunk, j = it - u * p.nchunk;
            const int lo = j * p.chunk_keys, hi = min(p.N, lo + p.chunk_keys);
            const int nt = (hi - lo + TN - 1) / TN;
            const int bprompt = u / units_per_prompt;
            const int2* pcs = p.pieces + (size_t)bprompt * p.P;
            int pi = p.chunk_first[(size_t)bprompt * p.cf_stride + j];
            const int pi_last = p.chunk_first[(size_t)bprompt * p.cf_stride + j + 1];
            // end of the current piece, and of the one after it: fetched one piece ahead so that the
            // load's latency never sits between a piece end and the next comparison
            int pend = pi < pi_last ? pcs[pi].y : 0x7fffffff;
            int pend_n = pi + 1 < pi_last ? pcs[pi + 1].y : 0x7fffffff;
            float m_ref = SHOTKV_NEG_INF, neg = 0.f;       // reference exponent of this (row, slice, item); neg = -m_ref
            float item_mm = SHOTKV_NEG_INF, item_zz = 0.f; // leader: the row's statistics over the item's pieces so far
            uint64_t z[2] = {0ull, 0ull};                  // four running sums of the current piece, as two packed pairs
            const int plain_end = min(hi, p.N - p.W + 1);  // keys below this count for every window row

            // piece `pi` is complete for this thread's columns.  A follower (slice > 0) posts its (m, z)
            // in the next slot of its ring; the leader (slice 0) collects one slot from every follower
            // of its rows, merges, and writes the piece's partials.
            auto flush = [&]() {
                float zz;
                {
                    float s0, s1, s2, s3;
                    tc::unpack2(z[0], s0, s1);
                    tc::unpack2(z[1], s2, s3);
                    zz = (s0 + s1) + (s2 + s3);
                }
                const int slot = nflush & (RD - 1);
                const uint32_t par = (uint32_t)(nflush / RD) & 1u;
                // out of range (or not a number): the exact kernel redoes the item.  Tested on this
                // slice's own sum, before any rescaling by another slice's reference could hide it.
                if (live && !(zz < tc::kRedoAbove)) {
                    p.redo[it] = 1;
                    *p.redo_any = 1;
                }
                if (slice != 0) {
                    const int ring = (blk * 4 + quad) * (NSL - 1) + (slice - 1);
                    const int rs = ring * RD + slot;
                    if (nflush >= RD) {                                   // the slot's previous contents must have been read
                        bool w = lane == 0 ? tc::mbar_wait(pp.extra_bar(rs * 2 + 1), par ^ 1u, pp.abort_flag, p.err, p.wait_cycles) : true;
                        w = __shfl_sync(0xffffffffu, w, 0);
                        __syncwarp();
                        ok = ok && w;
                    }
                    float2* dst = reinterpret_cast<float2*>(comb) + rs * 32 + lane;
                    *dst = make_float2(m_ref, zz);
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(pp.extra_bar(rs * 2));
                } else {
                    float mm = m_ref, ms[NSL > 1 ? NSL - 1 : 1], zs[NSL > 1 ? NSL - 1 : 1];
#pragma unroll
                    for (int s = 1; s < NSL; ++s) {
                        const int rs = ((blk * 4 + quad) * (NSL - 1) + (s - 1)) * RD + slot;
                        bool w = lane == 0 ? tc::mbar_wait(pp.extra_bar(rs * 2), par, pp.abort_flag, p.err, p.wait_cycles) : true;
                        w = __shfl_sync(0xffffffffu, w, 0);
                        __syncwarp();                                     // orders the other lanes' reads after lane 0's wait
                        ok = ok && w;
                        const float2 v = reinterpret_cast<const float2*>(comb)[rs * 32 + lane];
                        __syncwarp();
                        if (lane == 0) tc::mbar_arrive(pp.extra_bar(rs * 2 + 1));
                        ms[s - 1] = v.x;
                        zs[s - 1] = v.y;
                        mm = fmaxf(mm, v.x);
                    }
                    const float mu = mm == SHOTKV_NEG_INF ? 0.f : mm;
                    if (NSL > 1) zz *= ex2f(m_ref - mu);
#pragma unroll
                    for (int s = 1; s < NSL; ++s) zz += zs[s - 1] * ex2f(ms[s - 1] - mu);
                    // the merged reference is the larger of the slices' references, both fixed on the item's
                    // first tile: the same for every piece of the item, so only z goes out per piece
                    const size_t o = ((size_t)u * p.P + pi) * p.Rpad + row;
                    p.part_z[o] = live ? zz : 0.f;
                    {
                        const float mn = fmaxf(item_mm, mm);
                        const float mq = mn == SHOTKV_NEG_INF ? 0.f : mn;
                        item_zz = item_zz * ex2f(item_mm - mq) + zz * ex2f(mm - mq);
                        item_mm = mn;
                    }
                }
                z[0] = z[1] = 0ull;
                ++nflush;
                ++pi;
                pend = pend_n;
                pend_n = pi + 1 < pi_last ? pcs[pi + 1].y : 0x7fffffff;
            };

            // 32 columns starting at key kc0 that hold the end of the keys, the causal window, or a piece end
            auto chunk_slow = [&](uint32_t (&r)[32], int kc0) {
                while (pend <= kc0) flush();
                if (kc0 + 32 <= plain_end) {                             // every column counts; pieces end inside
                    tc::peel_chunk<PE>(r, scale, neg, mtab, kc0, pend, z, flush);
                    return;
                }
                const int lim = min(hi, plim + 1) - kc0;                 // columns of the chunk that count
                if (!__all_sync(0xffffffffu, lim >= 32)) tc::mask32(r, lim);
                tc::exp32(r, scale, neg);
                int start = 0;
                while (pend < kc0 + 32) {
                    const int e = pend - kc0;
                    z[0] = tc::fadd2(z[0], tc::pack2(tc::range32(r, start, e), 0.f));
                    start = e;
                    flush();
                }
                z[0] = tc::fadd2(z[0], tc::pack2(tc::range32(r, start, 32), 0.f));
            };

            for (int t = 0; t < nt; ++t) {
                const uint32_t tph = acc ? tfphase1 : tfphase0;
                // usually ready: one test by the whole warp, made uniform before anything depends on it
                if (!__all_sync(0xffffffffu, tc::mbar_try(pp.tfull(acc, blk), tph))) {
                    bool w = lane == 0 ? tc::mbar_wait(pp.tfull(acc, blk), tph, pp.abort_flag, p.err, p.wait_cycles) : true;   // one poller per warp
                    w = __shfl_sync(0xffffffffu, w, 0);
                    if (!w) ok = false;
                }
                if (!ok) break;
                if (acc) tfphase1 ^= 1; else tfphase0 ^= 1;
                tc::fence_after_sync();
                const int kc0 = lo + t * TN + slice * SLW;
                const uint32_t taddr = pp.tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)((acc * MB + blk) * TN + slice * SLW);
                uint32_t r[32];
                if (t == 0) {
                    // the item's reference exponent: this thread's maximum over its slice of the first tile
                    float cm = SHOTKV_NEG_INF;
#pragma unroll 1
                    for (int c = 0; c < NCH; ++c) {
                        tc::tmem_ld32_sync(r, taddr + c * 32);
                        const int lim = min(hi, plim + 1) - (kc0 + c * 32);
                        if (!__all_sync(0xffffffffu, lim >= 32)) tc::mask32(r, lim);
                        cm = fmaxf(cm, tc::max32(r));
                    }
                    if (cm != SHOTKV_NEG_INF) {
                        m_ref = fmaf(cm, scale, tc::kRefShift);
                        neg = -m_ref;
                    }
                }
                auto release = [&]() {                                   // this tile's accumulators are all in registers
                    tc::fence_before_sync();
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(pp.tempty(acc, blk));
                };
                if (kc0 + SLW <= min(pend, plain_end)) {
                    // most tiles: every column of the slice counts for every row (it lies before the
                    // item's end and before the first window position) and no piece ends inside it.
                    // One short loop without further branches.
#pragma unroll 1
                    for (int c = 0; c < NCH; ++c) {
                        tc::tmem_ld32_sync(r, taddr + c * 32);
                        tc::expacc32<PE>(r, scale, neg, z);
                    }
                    release();
                } else {
#pragma unroll 1
                    for (int c = 0; c < NCH; ++c) {
                        tc::tmem_ld32_sync(r, taddr + c * 32);
                        if (c == NCH - 1) release();
                        if (kc0 + c * 32 + 32 <= min(pend, plain_end)) tc::expacc32<PE>(r, scale, neg, z);
                        else chunk_slow(r, kc0 + c * 32);
                    }
                }
                acc ^= 1;
            }
            if (!ok) break;
            while (pi < pi_last) flush();
            if (slice == 0) {
                p.item_m[(size_t)it * p.Rpad + row] = live ? item_mm : 0.f;
                p.item_z[(size_t)it * p.Rpad + row] = live ? item_zz : 0.f;
            }
        }
    }

    tc::fence_before_sync();
    __syncthreads();
    tc::stamp(p.clk, 1);
    if (warp == 0) {
        __syncwarp();
        tc::fence_after_sync();
        tc::tmem_dealloc(pp.tmem_base, 512);
    }
}

}  // namespace shotkv
