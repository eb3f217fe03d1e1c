// Window attention scoring for units of more than 128 window rows (two 128-row blocks of Q), the
// kernel the prefill path runs first on them: the TMA producer, MMA issuers, work items and
// per-(piece, window row) outputs (m, z) of score_tc.cuh, the fixed reference exponent with
// exact-kernel repair and the two-pipe exponentials of score_fast.cuh, and an epilogue that never
// waits for tensor memory.
//
// Eight epilogue warps, one per (row block, tensor-memory lane quarter); a thread is one whole
// window row, so a piece's z (and the item's reference m) is written by one thread with no exchange.  The accumulator
// columns of the next 32-column chunk -- of the next tile too, once its barrier is seen complete
// -- are requested into a second set of registers before the arithmetic of the current chunk
// starts, so the load's latency runs beside the exponentials.  Where a piece ends inside a chunk
// the chunk's exponentials are split between the two pieces by multiplying with 0/1 masks read
// from a shared-memory table (one packed multiply-add per column pair and piece), which costs
// half the instructions of a predicated addition per column.
//
// What bounds this kernel on a B200 held at a 1 kW power cap is energy per tile, not a pipe: its
// epilogue takes the same cycles per tile with or without the MMAs running beside it, but the GPU
// settles near 1.5 GHz with them and at its full 1.96 GHz without.  The polynomial costs 5.5 issue
// slots per logit against 2 for the special-function path, so a larger share on the FMA pipe
// (PE of every 16 column pairs) saves cycles and spends energy; measured at the cap, shares from 2
// to 5 of 16 come out within the noise of the power controller, and below the cap the larger
// share is faster.
#pragma once
#include "score_fast.cuh"

namespace shotkv {

template <int D>
struct ScoreStreamCfg {
    static constexpr int kSub = D / 64;
    static constexpr int kSubBytes = 128 * 128;
    static constexpr int kQBytes = 2 * kSub * kSubBytes;
    static constexpr int kStageBytes = kSub * kSubBytes;
    static constexpr int kStages = D == 128 ? 4 : 6;
    static constexpr int kBarBytes = 1024;
    static constexpr int kCombBytes = tc::kSplitMaskBytes;     // split masks: [columns of the piece that ends][column pair] float4
    static constexpr int kSmemBytes = kQBytes + kStages * kStageBytes + kBarBytes + kCombBytes + 1024;
    static constexpr int kEpiWarps = 8;
    static constexpr int kThreads = 128 + kEpiWarps * 32;      // producer, two MMA issuers, one idle warp; epilogue
};

namespace tc {

// 32 consecutive fp32 columns of this thread's tensor-memory lane, requested but not waited for:
// the registers are not defined until tmem_ld_wait has been passed with the same array.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t (&v)[32], uint32_t taddr) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
// Waits for every tensor-memory load this thread has requested.  The array is passed as a
// read-write operand so that no use of its registers can be moved above the wait.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.wait::ld.sync.aligned;"
        : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]), "+r"(v[8]),
          "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]), "+r"(v[16]),
          "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]), "+r"(v[24]),
          "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
        :
        : "memory");
}

}  // namespace tc

template <int D, int PE>
__global__ void __launch_bounds__(ScoreStreamCfg<D>::kThreads, 1)
    score_stream_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const int q_box_rows,
                        const int k_box_rows, const ScoreTcParams p) {
    using Cfg = ScoreStreamCfg<D>;
    constexpr int TN = tc::kTileKeys, MB = 2;
    extern __shared__ unsigned char smem_raw[];
    tc::stamp(p.clk, 0);
    tc::Pipe<Cfg> pp;
    tc::pipe_setup(pp, smem_raw, 4, 0, 2);
    float4* mtab = reinterpret_cast<float4*>(tc::pipe_scratch(pp, smem_raw));   // split masks
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
        // a warp may touch the 32 tensor-memory lanes given by its index modulo 4
        const int blk = (warp - 4) >> 2, quad = warp & 3;  // 128-row block of Q, lane quarter
        const int row = blk * 128 + quad * 32 + lane;
        const bool live = row < p.R;                       // padding rows: their Q was never loaded
        const int plim = live ? p.N - p.W + (row % p.W) : p.N - 1;
        const float scale = p.scale_log2;
        const int units_per_prompt = p.L * p.Hkv;
        const uint32_t tlane = pp.tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(blk * TN);
        int tiles_before = 0;                              // tiles of earlier items (fixes the accumulator buffer of every tile)
        uint32_t tfphase0 = 0, tfphase1 = 0;
        bool ok = true;
        uint32_t ra[32], rb[32];                           // even and odd chunks of a tile
        for (int it = item_begin; it < item_end && ok; ++it) {
            const int u = it / p.nchunk, j = it - u * p.nchunk;
            const int lo = j * p.chunk_keys, hi = min(p.N, lo + p.chunk_keys);
            const int nt = max(0, (hi - lo + TN - 1) / TN);
            const int bprompt = u / units_per_prompt;
            const int2* pcs = p.pieces + (size_t)bprompt * p.P;
            int pi = p.chunk_first[(size_t)bprompt * p.cf_stride + j];
            const int pi_last = p.chunk_first[(size_t)bprompt * p.cf_stride + j + 1];
            // end of the current piece, and of the one after it (fetched one piece ahead)
            int pend = pi < pi_last ? pcs[pi].y : 0x7fffffff;
            int pend_n = pi + 1 < pi_last ? pcs[pi + 1].y : 0x7fffffff;
            float m_ref = SHOTKV_NEG_INF, neg = 0.f;       // reference exponent of this (row, item); neg = -m_ref
            uint64_t z[2] = {0ull, 0ull};                  // four running sums of the current piece, as two packed pairs
            const int plain_end = min(hi, p.N - p.W + 1);  // keys below this count for every window row
            float* out_z = p.part_z + ((size_t)u * p.P + pi) * p.Rpad + row;
            float zsum = 0.f;                              // sum of the item's pieces so far (they share m_ref)

            // piece `pi` is complete: write its partials and move on to the next piece
            auto flush = [&]() {
                float s0, s1, s2, s3;
                tc::unpack2(z[0], s0, s1);
                tc::unpack2(z[1], s2, s3);
                const float zz = (s0 + s1) + (s2 + s3);
                // out of range (or not a number): the exact kernel redoes the item
                if (live && !(zz < tc::kRedoAbove)) {
                    p.redo[it] = 1;
                    *p.redo_any = 1;
                }
                *out_z = live ? zz : 0.f;
                out_z += p.Rpad;
                zsum += zz;
                z[0] = z[1] = 0ull;
                ++pi;
                pend = pend_n;
                pend_n = pi + 1 < pi_last ? pcs[pi + 1].y : 0x7fffffff;
            };

            // 32 columns starting at key kc that hold the end of the keys, the causal window, or a piece end
            auto chunk_slow = [&](uint32_t (&r)[32], int kc) {
                while (pend <= kc) flush();
                if (kc + 32 <= plain_end) {                              // every column counts; pieces end inside
                    tc::peel_chunk<PE>(r, scale, neg, mtab, kc, pend, z, flush);
                    return;
                }
                const int lim = min(hi, plim + 1) - kc;                  // columns of the chunk that count
                if (!__all_sync(0xffffffffu, lim >= 32)) tc::mask32(r, lim);
                tc::exp32(r, scale, neg);
                int start = 0;
                while (pend < kc + 32) {
                    const int e = pend - kc;
                    z[0] = tc::fadd2(z[0], tc::pack2(tc::range32(r, start, e), 0.f));
                    start = e;
                    flush();
                }
                z[0] = tc::fadd2(z[0], tc::pack2(tc::range32(r, start, 32), 0.f));
            };
            auto chunk = [&](uint32_t (&r)[32], int kc) {
                if (kc + 32 <= min(pend, plain_end)) tc::expacc32<PE>(r, scale, neg, z);
                else chunk_slow(r, kc);
            };
            // waits (bounded) until the accumulators of the tile in buffer `a` are complete
            auto wait_tile = [&](int a) {
                const uint32_t tph = a ? tfphase1 : tfphase0;
                // usually ready: one test by the whole warp, made uniform before anything depends on it
                if (!__all_sync(0xffffffffu, tc::mbar_try(pp.tfull(a, blk), tph))) {
                    bool w = lane == 0 ? tc::mbar_wait(pp.tfull(a, blk), tph, pp.abort_flag, p.err, p.wait_cycles) : true;   // one poller per warp
                    w = __shfl_sync(0xffffffffu, w, 0);
                    if (!w) ok = false;
                }
                if (a) tfphase1 ^= 1; else tfphase0 ^= 1;
                tc::fence_after_sync();
            };

            bool have_a = false;                            // chunk 0 of the next tile has been requested into ra
            if (nt > 0) {
                // the reference exponent: this thread's maximum over the item's first tile
                const int a = tiles_before & 1;
                wait_tile(a);
                if (ok) {
                    const uint32_t taddr = tlane + (uint32_t)(a * MB * TN);
                    float cm = SHOTKV_NEG_INF;
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        tc::tmem_ld32_sync(ra, taddr + c * 32);
                        const int lim = min(hi, plim + 1) - (lo + c * 32);
                        if (!__all_sync(0xffffffffu, lim >= 32)) tc::mask32(ra, lim);
                        cm = fmaxf(cm, tc::max32(ra));
                    }
                    if (cm != SHOTKV_NEG_INF) {
                        m_ref = fmaf(cm, scale, tc::kRefShift);
                        neg = -m_ref;
                    }
                    tc::tmem_ld32_issue(ra, taddr);
                    have_a = true;
                }
            }
            for (int t = 0; t < nt && ok; ++t) {
                const int a = (tiles_before + t) & 1;
                const int kc0 = lo + t * TN;
                const uint32_t taddr = tlane + (uint32_t)(a * MB * TN);
                if (!have_a) {                              // the barrier was not complete when the previous tile looked
                    wait_tile(a);
                    if (!ok) break;
                    tc::tmem_ld32_issue(ra, taddr);
                }
                tc::tmem_ld_wait(ra);
                tc::tmem_ld32_issue(rb, taddr + 32);
                chunk(ra, kc0);
                tc::tmem_ld_wait(rb);
                tc::tmem_ld32_issue(ra, taddr + 64);
                chunk(rb, kc0 + 32);
                tc::tmem_ld_wait(ra);
                tc::tmem_ld32_issue(rb, taddr + 96);
                chunk(ra, kc0 + 64);
                tc::tmem_ld_wait(rb);
                // all of this tile's accumulators are in registers: hand the buffer back
                tc::fence_before_sync();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(pp.tempty(a, blk));
                // request the first chunk of the next tile if its accumulators are complete already
                have_a = false;
                if (t + 1 < nt) {
                    const int an = a ^ 1;
                    const uint32_t tph = an ? tfphase1 : tfphase0;
                    if (__all_sync(0xffffffffu, tc::mbar_try(pp.tfull(an, blk), tph))) {
                        if (an) tfphase1 ^= 1; else tfphase0 ^= 1;
                        tc::fence_after_sync();
                        tc::tmem_ld32_issue(ra, tlane + (uint32_t)(an * MB * TN));
                        have_a = true;
                    }
                }
                chunk(rb, kc0 + 96);
            }
            if (!ok) break;
            while (pi < pi_last) flush();
            // the row's statistics over the whole item: its reference and the sum of its pieces
            p.item_m[(size_t)it * p.Rpad + row] = live ? m_ref : 0.f;
            p.item_z[(size_t)it * p.Rpad + row] = live ? zsum : 0.f;
            tiles_before += nt;
        }
        // an abort may leave a requested chunk unread: nothing of tensor memory is in flight past here
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
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
