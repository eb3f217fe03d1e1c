// Window attention scoring on the 5th-generation tensor cores (tcgen05.mma, accumulators in
// tensor memory) with K streamed by TMA: the STATS pass of the scoring step.
//
// Persistent CTAs, one per SM, each owning a contiguous range of (unit, piece) work items
// (unit = prompt x layer x kv head; a piece is a key range of at most 512 keys that never
// straddles a shot boundary).  Warp roles:
//   warp 0      TMA producer: the unit's window queries Q (once per unit) and K tiles of 128 keys
//               into a ring of 128-byte-swizzled shared-memory stages
//   warp 1      MMA issuer: S[128 x 128] = Q_block . K_tile^T per 128-row block of Q, fp32
//               accumulators double-buffered in tensor memory
//   warp 2      tensor-memory allocation
//   warps 4-11  epilogue: one thread per window row; reads its row of S from tensor memory and
//               keeps, per piece, a reference maximum m and z = sum exp2(x - m)
// Per (piece, row) the pair (m, z) goes to global memory; the reductions over pieces, rows and
// heads that turn them into shot scores are done by the kernels in score_mma.cuh.
//
// Every wait on an mbarrier is bounded: after about two seconds a waiter raises the CTA's abort
// flag and the device error word, all roles leave their loops, outstanding bulk copies are
// waited for (bounded again), tensor memory is released and the kernel returns.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace shotkv {

struct ScoreTcParams {
    const int2* pieces;   // [B][P] key ranges [lo, hi)
    int P;                // pieces per prompt
    int L, Hkv, N, W, R, Rpad;
    int total_items;      // U * P
    float scale_log2;     // log2(e)/sqrt(d)
    float* part_m;        // [U][P][Rpad]
    float* part_z;        // [U][P][Rpad]
    int* err;             // error word (host-visible); set to 1 when a bounded wait gave up
};

template <int D, int MB>
struct ScoreTcCfg {
    static constexpr int kSub = D / 64;                    // 64-element (128-byte) sub-tiles per row
    static constexpr int kSubBytes = 128 * 128;            // 128 rows x 128 bytes
    static constexpr int kQBytes = MB * kSub * kSubBytes;
    static constexpr int kStageBytes = kSub * kSubBytes;
    static constexpr int kStages = D == 128 ? (MB == 2 ? 4 : 5) : 6;
    static constexpr int kBarBytes = 1024;
    static constexpr int kSmemBytes = kQBytes + kStages * kStageBytes + kBarBytes + 2 * 128 * 2 * 4 + 1024;
};

namespace tc {

constexpr int kTileKeys = 128;
constexpr long long kWaitCycles = 4000000000LL;   // about two seconds

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    return done != 0;
}
// Bounded wait.  Returns false when the CTA is aborting (this waiter gave up, or another did).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* err) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try(bar, parity)) return true;
        if ((spin & 63u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > kWaitCycles) {
                *abort_flag = 1;
                atomicExch(err, 1);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t slot, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem desc] . B[smem desc]^T, bf16 x bf16 -> fp32, one CTA.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrives once on `bar` when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Shared-memory operand descriptor: K-major rows of 128 bytes, 128-byte swizzle, 8-row groups
// 1024 bytes apart (the layout TMA writes with CU_TENSOR_MAP_SWIZZLE_128B).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

// 32 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld32(uint32_t (&v)[32], uint32_t taddr) {
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
// Waits for this thread's tensor-memory loads.  The registers are named as in/out operands so
// that no use of them can be scheduled before the wait.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&v)[32]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                   "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]),
                   "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]),
                   "+r"(v[23]), "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]),
                   "+r"(v[30]), "+r"(v[31])
                 :
                 : "memory");
}

// One 32-column chunk of a row: mask, refresh the reference maximum if the chunk exceeds it by
// more than 2^8, add exp2(x*scale - m) to the running sum.  `valid` = columns of the chunk that
// count (<= 0: none, >= 32: all).
__device__ __forceinline__ void row_chunk(uint32_t (&raw)[32], int valid, float scale, float& m_ref, float& z) {
    float v[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(raw[i]);
    if (!__all_sync(0xffffffffu, valid >= 32)) {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = i < valid ? v[i] : SHOTKV_NEG_INF;
    }
    float c0 = fmaxf(v[0], v[1]), c1 = fmaxf(v[2], v[3]), c2 = fmaxf(v[4], v[5]), c3 = fmaxf(v[6], v[7]);
#pragma unroll
    for (int i = 8; i < 32; i += 8) {
        c0 = fmaxf(c0, fmaxf(v[i], v[i + 1]));
        c1 = fmaxf(c1, fmaxf(v[i + 2], v[i + 3]));
        c2 = fmaxf(c2, fmaxf(v[i + 4], v[i + 5]));
        c3 = fmaxf(c3, fmaxf(v[i + 6], v[i + 7]));
    }
    const float cm = fmaxf(fmaxf(c0, c1), fmaxf(c2, c3)) * scale;
    if (cm > m_ref + 8.f) {            // also taken the first time (m_ref = -inf, z = 0)
        z *= ex2f(m_ref - cm);
        m_ref = cm;
    }
    const float neg = m_ref == SHOTKV_NEG_INF ? 0.f : -m_ref;
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        s0 += ex2f(fmaf(v[i], scale, neg));
        s1 += ex2f(fmaf(v[i + 1], scale, neg));
        s2 += ex2f(fmaf(v[i + 2], scale, neg));
        s3 += ex2f(fmaf(v[i + 3], scale, neg));
    }
    z += (s0 + s1) + (s2 + s3);
}

}  // namespace tc

template <int D, int MB>
__global__ void __launch_bounds__(384, 1) score_tc_kernel(const __grid_constant__ CUtensorMap tmQ,
                                                         const __grid_constant__ CUtensorMap tmK, const int q_box_rows,
                                                         const int k_box_rows, const ScoreTcParams p) {
    using Cfg = ScoreTcCfg<D, MB>;
    constexpr int NSUB = Cfg::kSub, KSTEPS = D / 16, NST = Cfg::kStages, TN = tc::kTileKeys;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    unsigned char* gbase = smem_raw + (base - raw_addr);
    const uint32_t sQ = base, sK = base + Cfg::kQBytes, sBar = sK + NST * Cfg::kStageBytes;
    auto bar_full = [&](int s) { return sBar + 8u * s; };
    auto bar_empty = [&](int s) { return sBar + 8u * (NST + s); };
    const uint32_t bar_qfull = sBar + 8u * (2 * NST), bar_qempty = bar_qfull + 8u;
    auto bar_tfull = [&](int a) { return sBar + 8u * (2 * NST + 2 + a); };
    auto bar_tempty = [&](int a) { return sBar + 8u * (2 * NST + 4 + a); };
    const uint32_t tmem_slot = sBar + 8u * (2 * NST + 6);
    volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(gbase + (tmem_slot - base));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + (tmem_slot - base) + 4);
    float* comb = reinterpret_cast<float*>(gbase + (sBar - base) + Cfg::kBarBytes);   // [2][128][2], MB == 1 only

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < NST; ++s) {
            tc::mbar_init(bar_full(s), 1);
            tc::mbar_init(bar_empty(s), 1);
        }
        tc::mbar_init(bar_qfull, 1);
        tc::mbar_init(bar_qempty, 1);
        for (int a = 0; a < 2; ++a) {
            tc::mbar_init(bar_tfull(a), 1);
            tc::mbar_init(bar_tempty(a), 8);      // one arrival per epilogue warp
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        tc::tmem_alloc(tmem_slot, 512);
        tc::tmem_relinquish();
    }
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    const uint32_t tmem_base = *tmem_slot_g;

    const long long total = p.total_items;
    const int item_begin = (int)(total * blockIdx.x / gridDim.x);
    const int item_end = (int)(total * (blockIdx.x + 1) / gridDim.x);
    const int units_per_prompt = p.L * p.Hkv;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0, cur_u = -1, outstanding = 0;
            uint32_t ephase = 1, qephase = 1;
            bool ok = true;
            for (int it = item_begin; it < item_end && ok; ++it) {
                const int u = it / p.P, pc = it - u * p.P;
                const int2 r = p.pieces[(size_t)(u / units_per_prompt) * p.P + pc];
                const int nt = (r.y - r.x + TN - 1) / TN;
                if (nt <= 0) continue;
                if (u != cur_u) {
                    if (!(ok = tc::mbar_wait(bar_qempty, qephase, abort_flag, p.err))) break;
                    qephase ^= 1;
                    tc::mbar_expect_tx(bar_qfull, MB * NSUB * q_box_rows * 128);
#pragma unroll
                    for (int j = 0; j < MB; ++j)
#pragma unroll
                        for (int sub = 0; sub < NSUB; ++sub)
                            tc::tma_load_2d(sQ + (j * NSUB + sub) * Cfg::kSubBytes, &tmQ, sub * 64, u * p.R + j * 128, bar_qfull);
                    cur_u = u;
                }
                for (int t = 0; t < nt; ++t) {
                    if (!(ok = tc::mbar_wait(bar_empty(stage), ephase, abort_flag, p.err))) break;
                    tc::mbar_expect_tx(bar_full(stage), NSUB * k_box_rows * 128);
#pragma unroll
                    for (int sub = 0; sub < NSUB; ++sub)
                        tc::tma_load_3d(sK + stage * Cfg::kStageBytes + sub * Cfg::kSubBytes, &tmK, sub * 64, r.x + t * TN, u,
                                        bar_full(stage));
                    outstanding = outstanding < NST ? outstanding + 1 : NST;
                    if (++stage == NST) {
                        stage = 0;
                        ephase ^= 1;
                    }
                }
            }
            if (!ok) {
                // aborting: give the copies already issued a bounded time to land before the CTA ends
                const long long t0 = clock64();
                int s = stage;
                uint32_t ph = ephase;
                for (int k = 0; k < outstanding; ++k) {
                    if (--s < 0) {
                        s = NST - 1;
                        ph ^= 1;
                    }
                    while (!tc::mbar_try(bar_full(s), ph ^ 1) && clock64() - t0 < tc::kWaitCycles) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TN >> 3) << 17) | ((128u >> 4) << 24);
            int stage = 0, acc = 0, cur_u = -1;
            uint32_t fphase = 0, qfphase = 0, tephase[2] = {1, 1};
            bool ok = true;
            for (int it = item_begin; it < item_end && ok; ++it) {
                const int u = it / p.P, pc = it - u * p.P;
                const int2 r = p.pieces[(size_t)(u / units_per_prompt) * p.P + pc];
                const int nt = (r.y - r.x + TN - 1) / TN;
                if (nt <= 0) continue;
                if (u != cur_u) {
                    if (cur_u >= 0) tc::umma_commit(bar_qempty);     // Q may be replaced once these MMAs are done
                    if (!(ok = tc::mbar_wait(bar_qfull, qfphase, abort_flag, p.err))) break;
                    qfphase ^= 1;
                    cur_u = u;
                }
                for (int t = 0; t < nt; ++t) {
                    if (!(ok = tc::mbar_wait(bar_full(stage), fphase, abort_flag, p.err))) break;
                    if (!(ok = tc::mbar_wait(bar_tempty(acc), tephase[acc], abort_flag, p.err))) break;
                    tephase[acc] ^= 1;
                    tc::fence_after_sync();
                    const uint32_t kb = sK + stage * Cfg::kStageBytes;
#pragma unroll
                    for (int j = 0; j < MB; ++j) {
                        const uint32_t d_tmem = tmem_base + (uint32_t)((acc * MB + j) * TN);
#pragma unroll
                        for (int ks = 0; ks < KSTEPS; ++ks) {
                            const uint32_t a_addr = sQ + (j * NSUB + (ks >> 2)) * Cfg::kSubBytes + (ks & 3) * 32;
                            const uint32_t b_addr = kb + (ks >> 2) * Cfg::kSubBytes + (ks & 3) * 32;
                            tc::umma_bf16(d_tmem, tc::smem_desc(a_addr), tc::smem_desc(b_addr), idesc, ks > 0);
                        }
                    }
                    tc::umma_commit(bar_empty(stage));
                    tc::umma_commit(bar_tfull(acc));
                    if (++stage == NST) {
                        stage = 0;
                        fphase ^= 1;
                    }
                    acc ^= 1;
                }
            }
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ epilogue
        const int wg = (warp - 4) >> 2, quad = warp & 3;
        const int blk = MB == 2 ? wg : 0;                 // 128-row block of Q this warpgroup reads
        const int col_base = MB == 2 ? 0 : wg * 64;       // MB == 1: the two warpgroups split the columns
        constexpr int NCH = MB == 2 ? 4 : 2;
        const int row = blk * 128 + quad * 32 + lane;
        const int plim = row < p.R ? p.N - p.W + (row % p.W) : p.N - 1;
        int acc = 0, item_no = 0;
        uint32_t tfphase[2] = {0, 0};
        bool ok = true;
        for (int it = item_begin; it < item_end && ok; ++it, ++item_no) {
            const int u = it / p.P, pc = it - u * p.P;
            const int2 r = p.pieces[(size_t)(u / units_per_prompt) * p.P + pc];
            const int nt = (r.y - r.x + TN - 1) / TN;
            float m_ref = SHOTKV_NEG_INF, z = 0.f;
            for (int t = 0; t < nt; ++t) {
                ok = tc::mbar_wait(bar_tfull(acc), tfphase[acc], abort_flag, p.err);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tfphase[acc] ^= 1;
                tc::fence_after_sync();
                const int key0 = r.x + t * TN;
                const int lim = min(r.y - key0, plim + 1 - key0) - col_base;     // valid columns from col_base on
                const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)((acc * MB + blk) * TN + col_base);
                uint32_t va[32], vb[32];
                tc::tmem_ld32(va, taddr);
#pragma unroll
                for (int c = 0; c < NCH; c += 2) {
                    tc::tmem_ld_wait(va);
                    tc::tmem_ld32(vb, taddr + (c + 1) * 32);
                    tc::row_chunk(va, lim - c * 32, p.scale_log2, m_ref, z);
                    tc::tmem_ld_wait(vb);
                    if (c + 2 < NCH) {
                        tc::tmem_ld32(va, taddr + (c + 2) * 32);
                    } else {
                        // this tile's accumulators are in registers: hand the buffer back
                        tc::fence_before_sync();
                        __syncwarp();
                        if (lane == 0) tc::mbar_arrive(bar_tempty(acc));
                    }
                    tc::row_chunk(vb, lim - (c + 1) * 32, p.scale_log2, m_ref, z);
                }
                acc ^= 1;
            }
            if (!ok) break;
            const size_t o = ((size_t)u * p.P + pc) * p.Rpad + row;
            if (row >= p.R) {          // padding row: its Q rows were never loaded; keep the partials finite
                m_ref = 0.f;
                z = 0.f;
            }
            if (MB == 2) {
                p.part_m[o] = m_ref;
                p.part_z[o] = z;
            } else {
                float* cb = comb + (item_no & 1) * 256 + (quad * 32 + lane) * 2;
                if (wg == 1) {
                    cb[0] = m_ref;
                    cb[1] = z;
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (wg == 0) {
                    const float m1 = cb[0], z1 = cb[1];
                    const float mm = fmaxf(m_ref, m1);
                    const float mu = mm == SHOTKV_NEG_INF ? 0.f : mm;
                    p.part_m[o] = mm;
                    p.part_z[o] = z * ex2f(m_ref - mu) + z1 * ex2f(m1 - mu);
                }
            }
        }
    }

    tc::fence_before_sync();
    __syncthreads();
    if (warp == 2) {
        tc::fence_after_sync();
        tc::tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace shotkv
