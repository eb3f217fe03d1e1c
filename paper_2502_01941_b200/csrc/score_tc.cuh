// Window attention scoring on the 5th-generation tensor cores (tcgen05.mma, accumulators in
// tensor memory) with K streamed by TMA: the exact scoring kernel (a running maximum per row),
// and the parts every tensor-core pass of this library shares -- PTX wrappers, the shared-memory
// and barrier map (tc::Pipe), the TMA producer and the MMA issuer (tc::producer_role,
// tc::mma_role).  The prefill path runs score_fast.cuh first and this kernel as its repair
// launch; with SHOTKV_SCORING_EXACT this kernel does all the work.
//
// Persistent CTAs, one per SM, each owning a contiguous range of work items.  An item is one
// (unit, chunk): unit = prompt x layer x kv head, chunk = a run of whole 128-key tiles of that
// unit's keys.  Chunk ends and shot boundaries cut the keys into "pieces"; per (piece, window
// row) the kernel emits a reference maximum m and z = sum exp2(x - m) over the piece's keys.
// Warp roles:
//   warp 0      tensor-memory allocation; TMA producer: the unit's window queries Q (once per unit) and K tiles of 128 keys
//               into a ring of 128-byte-swizzled shared-memory stages
//   warp 1      MMA issuer: S[128 x 128] = Q_block . K_tile^T per 128-row block of Q, fp32
//               accumulators double-buffered in tensor memory
//   warps 4-19  epilogue: every thread owns one window row and a slice of a tile's columns (64
//               of 128 when there are two row blocks, 32 when there is one), walks them in
//               chunks of 32 registers, and splits its running sum wherever a piece ends inside
//               a chunk.  The slices of a row are merged through shared memory when a piece is
//               complete, in a fixed order.
// The reductions over pieces, rows and heads that turn (m, z) into shot scores are done by the
// kernels in reductions.cuh.
//
// Every wait on an mbarrier is bounded: after about two seconds a waiter raises the CTA's abort
// flag and the device error word, all roles leave their loops, outstanding bulk copies are
// waited for (bounded again), tensor memory is released and the kernel returns.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace shotkv {

struct ScoreTcParams {
    const int2* pieces;       // [B][P] key ranges [lo, hi), ascending, covering [0, N)
    const int* chunk_first;   // [B][cf_stride] index of the first piece of every chunk (nchunk + 1 used)
    int cf_stride;
    int P;                    // pieces per prompt (row length of `pieces`)
    int nchunk, chunk_keys;   // chunks per unit; keys per chunk (a multiple of 128)
    int L, Hkv, N, W, R, Rpad;
    int total_items;          // U * nchunk
    float scale_log2;     // log2(e)/sqrt(d)
    float* part_m;        // [U][P][Rpad]  per-piece reference: written by the exact kernel only
    float* part_z;        // [U][P][Rpad]
    float* item_m;        // [U * nchunk][Rpad]  the one reference of an item's pieces, and the sum of their z:
    float* item_z;        //                     written by the kernels that fix a reference per item
    int* err;             // error word (host-visible); set to 1 when a bounded wait gave up
    long long wait_cycles;    // limit of every bounded wait, in SM clock cycles
    long long* clk;           // optional (host-visible): SM cycle counter and nanosecond timer of CTA 0 at kernel start and end
    // Item filter.  The fast kernel (score_fast.cuh) raises redo[item] and *redo_any when an item's
    // sums left the fp32 range it works in; the exact kernel, given the same arrays, recomputes
    // only those items and returns at once when there is none.  Both NULL: every item is done.
    int* redo;            // [total_items]
    int* redo_any;
    int* repaired;        // host-visible count of items recomputed under the filter (diagnostic)
};

template <int D, int MB>
struct ScoreTcCfg {
    static constexpr int kSub = D / 64;                    // 64-element (128-byte) sub-tiles per row
    static constexpr int kSubBytes = 128 * 128;            // 128 rows x 128 bytes
    static constexpr int kQBytes = MB * kSub * kSubBytes;
    static constexpr int kStageBytes = kSub * kSubBytes;
    static constexpr int kStages = D == 128 ? (MB == 2 ? 4 : 5) : 6;
    static constexpr int kBarBytes = 1024;
    static constexpr int kCombBytes = 2 * 4 * 128 * 2 * 4;   // [parity][slice][row][m, z]
    static constexpr int kSmemBytes = kQBytes + kStages * kStageBytes + kBarBytes + kCombBytes + 1024;
    static constexpr int kSlices = 4 / MB;                    // column slices of a tile, one per epilogue warpgroup
    static constexpr int kThreads = 128 + 16 * 32;            // producer, MMA issuer, two idle warps; 16 epilogue warps
};

namespace tc {

constexpr int kTileKeys = 128;
constexpr long long kWaitCycles = 4000000000LL;   // default limit of a bounded wait: about two seconds

// Diagnostic: CTA 0's SM cycle counter and the global nanosecond timer, written to clk[2*which] and
// clk[2*which + 1] (which = 0 at kernel start, 1 at its end).  Their quotient is the SM clock the
// kernel really ran at, which under a power cap is not the clock a sampler reads between kernels.
__device__ __forceinline__ void stamp(long long* clk, int which) {
    if (clk && blockIdx.x == 0 && threadIdx.x == 0) {
        unsigned long long ns;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));
        clk[2 * which] = clock64();
        clk[2 * which + 1] = (long long)ns;
    }
}
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
// Bounded wait: gives up after `limit` cycles.  Returns false when the CTA is aborting (this
// waiter gave up, or another did); the waiter that gives up raises the CTA's abort flag and the
// device error word.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* err, long long limit) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try(bar, parity)) return true;
        if ((spin & 63u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > limit) {
                *abort_flag = 1;
                atomicExch(err, 1);
                return false;
            }
        }
    }
}

// try_wait that lets the hardware suspend the thread until the phase completes or about `ns`
// nanoseconds have passed, whichever comes first.
__device__ __forceinline__ bool mbar_try_suspend(uint32_t bar, uint32_t parity, uint32_t ns) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity), "r"(ns)
        : "memory");
    return done != 0;
}
// The same for the single-thread producer and MMA roles, which wait long and often.  They wait
// suspended inside try_wait (up to a microsecond at a time) instead of polling: a polling loop with
// short sleeps executed about 110 iterations per tile between the three of them, an eighth of all
// the warp instructions of the kernel, in issue slots and power the epilogue warps need.
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* err, long long limit) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_suspend(bar, parity, 1000u)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > limit) {
            *abort_flag = 1;
            atomicExch(err, 1);
            return false;
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

// 32 consecutive fp32 columns of this thread's tensor-memory lane, loaded and waited for in one
// statement, so that the registers are defined when it ends.
__device__ __forceinline__ void tmem_ld32_sync(uint32_t (&v)[32], uint32_t taddr) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
// ---- per-row arithmetic on 32 accumulator columns held in registers -----------------------
#define SKV_F(r, i) __uint_as_float((r)[i])

__device__ __forceinline__ float max32(const uint32_t (&r)[32]) {
    float c0 = fmaxf(SKV_F(r, 0), SKV_F(r, 1)), c1 = fmaxf(SKV_F(r, 2), SKV_F(r, 3));
    float c2 = fmaxf(SKV_F(r, 4), SKV_F(r, 5)), c3 = fmaxf(SKV_F(r, 6), SKV_F(r, 7));
#pragma unroll
    for (int i = 8; i < 32; i += 8) {
        c0 = fmaxf(c0, fmaxf(SKV_F(r, i), SKV_F(r, i + 1)));
        c1 = fmaxf(c1, fmaxf(SKV_F(r, i + 2), SKV_F(r, i + 3)));
        c2 = fmaxf(c2, fmaxf(SKV_F(r, i + 4), SKV_F(r, i + 5)));
        c3 = fmaxf(c3, fmaxf(SKV_F(r, i + 6), SKV_F(r, i + 7)));
    }
    return fmaxf(fmaxf(c0, c1), fmaxf(c2, c3));
}
// columns at or beyond `valid` become -inf
__device__ __forceinline__ void mask32(uint32_t (&r)[32], int valid) {
#pragma unroll
    for (int i = 0; i < 32; ++i)
        if (i >= valid) r[i] = 0xff800000u;
}
// Two fp32 values in one 64-bit register, for the packed fp32 instructions of sm_100.
__device__ __forceinline__ uint64_t pack2(float a, float b) {
    uint64_t v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(a), "f"(b));
    return v;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t fadd2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// sum of exp2(x*scale + neg).  The multiply-add and the accumulation run two columns per
// instruction: beside each exp2 on the special-function unit only about two and a half other
// instructions can issue, so every instruction per column counts.
__device__ __forceinline__ float expsum32(const uint32_t (&r)[32], float scale, float neg) {
    const uint64_t sc2 = pack2(scale, scale), ng2 = pack2(neg, neg);
    uint64_t a0 = pack2(0.f, 0.f), a1 = a0;
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        float x0, x1, x2, x3;
        unpack2(ffma2(pack2(SKV_F(r, i), SKV_F(r, i + 1)), sc2, ng2), x0, x1);
        unpack2(ffma2(pack2(SKV_F(r, i + 2), SKV_F(r, i + 3)), sc2, ng2), x2, x3);
        a0 = fadd2(a0, pack2(ex2f(x0), ex2f(x1)));
        a1 = fadd2(a1, pack2(ex2f(x2), ex2f(x3)));
    }
    float s0, s1, s2, s3;
    unpack2(a0, s0, s1);
    unpack2(a1, s2, s3);
    return (s0 + s1) + (s2 + s3);
}
// exp2(x*scale + neg) in place
__device__ __forceinline__ void exp32(uint32_t (&r)[32], float scale, float neg) {
#pragma unroll
    for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(ex2f(fmaf(SKV_F(r, i), scale, neg)));
}
__device__ __forceinline__ float sum32(const uint32_t (&e)[32]) {
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        s0 += SKV_F(e, i);
        s1 += SKV_F(e, i + 1);
        s2 += SKV_F(e, i + 2);
        s3 += SKV_F(e, i + 3);
    }
    return (s0 + s1) + (s2 + s3);
}
// lo = sum of e[i] for i < nb, hi = the rest (both summed directly: no subtraction of prefixes,
// so a tiny piece next to a dominant key keeps its own relative accuracy)
__device__ __forceinline__ void split32(const uint32_t (&e)[32], int nb, float& lo, float& hi) {
    float l0 = 0.f, l1 = 0.f, h0 = 0.f, h1 = 0.f;
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        if (i < nb) l0 += SKV_F(e, i); else h0 += SKV_F(e, i);
        if (i + 1 < nb) l1 += SKV_F(e, i + 1); else h1 += SKV_F(e, i + 1);
    }
    lo = l0 + l1;
    hi = h0 + h1;
}
// sum of e[i] for a <= i < b
__device__ __forceinline__ float range32(const uint32_t (&e)[32], int a, int b) {
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        s0 += (i >= a && i < b) ? SKV_F(e, i) : 0.f;
        s1 += (i + 1 >= a && i + 1 < b) ? SKV_F(e, i + 1) : 0.f;
    }
    return s0 + s1;
}



// ---- the parts both scoring kernels share: shared-memory map, TMA producer, MMA issuer -------
template <class Cfg>
struct Pipe {
    static constexpr int NST = Cfg::kStages;
    uint32_t sQ, sK, sBar;      // shared-memory addresses: window queries, K stage ring, barriers
    uint32_t tmem_base;
    volatile int* abort_flag;
    __device__ __forceinline__ uint32_t full(int s) const { return sBar + 8u * s; }
    __device__ __forceinline__ uint32_t empty(int s) const { return sBar + 8u * (NST + s); }
    __device__ __forceinline__ uint32_t qfull() const { return sBar + 8u * (2 * NST); }
    __device__ __forceinline__ uint32_t qempty() const { return sBar + 8u * (2 * NST + 1); }
    // accumulator-ready / accumulator-free barriers per (buffer, row block): the two row blocks of a
    // tile are handed over separately
    __device__ __forceinline__ uint32_t tfull(int a, int b) const { return sBar + 8u * (2 * NST + 2 + a * 2 + b); }
    __device__ __forceinline__ uint32_t tempty(int a, int b) const { return sBar + 8u * (2 * NST + 6 + a * 2 + b); }
    __device__ __forceinline__ uint32_t tmem_slot() const { return sBar + 8u * (2 * NST + 10); }
    __device__ __forceinline__ uint32_t extra_bar(int i) const { return sBar + 256u + 8u * i; }
};

// Barrier set-up, tensor-memory allocation and the CTA-wide hand-over of its address.  Called by
// every thread; `tempty_arrivals` = epilogue warps that release one (buffer, row block).
// `extra` further barriers of one arrival each are initialised from pp.extra_bar(0) on.
// `mma_threads` = threads running mma_role (each commits once to the Q-free barrier per unit).
template <class Cfg>
__device__ __forceinline__ void pipe_setup(Pipe<Cfg>& pp, unsigned char* smem_raw, int tempty_arrivals, int extra = 0,
                                           int mma_threads = 1) {
    constexpr int NST = Cfg::kStages;
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    unsigned char* gbase = smem_raw + (base - raw_addr);
    pp.sQ = base;
    pp.sK = base + Cfg::kQBytes;
    pp.sBar = pp.sK + NST * Cfg::kStageBytes;
    volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(gbase + (pp.tmem_slot() - base));
    pp.abort_flag = reinterpret_cast<volatile int*>(gbase + (pp.tmem_slot() - base) + 4);
    if (threadIdx.x == 0) {
        for (int s = 0; s < NST; ++s) {
            mbar_init(pp.full(s), 1);
            mbar_init(pp.empty(s), 1);
        }
        mbar_init(pp.qfull(), 1);
        mbar_init(pp.qempty(), mma_threads);
        for (int a = 0; a < 2; ++a)
            for (int b = 0; b < 2; ++b) {
                mbar_init(pp.tfull(a, b), 1);
                mbar_init(pp.tempty(a, b), tempty_arrivals);
            }
        for (int i = 0; i < extra; ++i) mbar_init(pp.extra_bar(i), 1);
        *pp.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if ((threadIdx.x >> 5) == 0) {
        tmem_alloc(pp.tmem_slot(), 512);
        tmem_relinquish();
    }
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    pp.tmem_base = *tmem_slot_g;
}
// The scratch area behind the barriers (merging of a row's column slices).
template <class Cfg>
__device__ __forceinline__ float* pipe_scratch(const Pipe<Cfg>& pp, unsigned char* smem_raw) {
    const uint32_t raw_addr = smem_u32(smem_raw);
    return reinterpret_cast<float*>(smem_raw + (pp.sBar - raw_addr) + Cfg::kBarBytes);
}

// One thread: the unit's window queries (once per unit) and K tiles of 128 keys into the ring.
// FILTERED: skip the items whose redo flag is clear (the exact kernel's repair launches).
// QKMAJOR: lay Q out k-block major (all rows of one 64-element k block contiguous), as a B
// operand of more than 128 rows needs; otherwise row-block major (each 128-row block contiguous).
template <int D, int MB, bool FILTERED, bool QKMAJOR, class Cfg>
__device__ __forceinline__ void producer_role(const Pipe<Cfg>& pp, const CUtensorMap* tmQ, const CUtensorMap* tmK,
                                              int q_box_rows, int k_box_rows, const ScoreTcParams& p, int item_begin,
                                              int item_end) {
    constexpr int NSUB = Cfg::kSub, NST = Cfg::kStages, TN = kTileKeys;
    int stage = 0, cur_u = -1, outstanding = 0;
    uint32_t ephase = 1, qephase = 1;
    bool ok = true;
    for (int it = item_begin; it < item_end && ok; ++it) {
        if (FILTERED && p.redo && !p.redo[it]) continue;
        const int u = it / p.nchunk, j = it - u * p.nchunk;
        const int lo = j * p.chunk_keys, hi = min(p.N, lo + p.chunk_keys);
        const int nt = (hi - lo + TN - 1) / TN;
        if (nt <= 0) continue;
        if (u != cur_u) {
            if (!(ok = mbar_wait_relaxed(pp.qempty(), qephase, pp.abort_flag, p.err, p.wait_cycles))) break;
            qephase ^= 1;
            mbar_expect_tx(pp.qfull(), MB * NSUB * q_box_rows * 128);
#pragma unroll
            for (int b = 0; b < MB; ++b)
#pragma unroll
                for (int sub = 0; sub < NSUB; ++sub)
                    tma_load_2d(pp.sQ + (QKMAJOR ? sub * MB + b : b * NSUB + sub) * Cfg::kSubBytes, tmQ, sub * 64, u * p.R + b * 128,
                                pp.qfull());
            cur_u = u;
        }
        for (int t = 0; t < nt; ++t) {
            if (!(ok = mbar_wait_relaxed(pp.empty(stage), ephase, pp.abort_flag, p.err, p.wait_cycles))) break;
            mbar_expect_tx(pp.full(stage), NSUB * k_box_rows * 128);
#pragma unroll
            for (int sub = 0; sub < NSUB; ++sub)
                tma_load_3d(pp.sK + stage * Cfg::kStageBytes + sub * Cfg::kSubBytes, tmK, sub * 64, lo + t * TN, u, pp.full(stage));
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
            while (!mbar_try(pp.full(s), ph ^ 1) && clock64() - t0 < p.wait_cycles) {
            }
        }
    }
}

// S[128 x 128] = Q_block . K_tile^T per 128-row block of Q, fp32 accumulators double-buffered in
// tensor memory (buffer a, row block b at column (a * MB + b) * 128).  Run by NT threads of
// different warps; thread `which` issues the tiles whose running index is `which` modulo NT.
// With NT = 2 each thread owns one accumulator buffer, so the two never touch the same barriers
// except the K-stage ring (each waits for and frees the stages of its own tiles) and the Q pair.
// A lone issuing thread shares its scheduler with four epilogue warps that seldom stall, and is
// selected so rarely that sixteen MMAs per tile take it longer than the tile's epilogue.
template <int D, int MB, bool FILTERED, int NT, class Cfg>
__device__ __forceinline__ void mma_role(const Pipe<Cfg>& pp, const ScoreTcParams& p, int item_begin, int item_end,
                                         int which) {
    constexpr int NSUB = Cfg::kSub, KSTEPS = D / 16, NST = Cfg::kStages, TN = kTileKeys;
    constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TN >> 3) << 17) | ((128u >> 4) << 24);
    // a thread that met a stage only every other turn of the ring would wait on a parity the barrier may
    // already have passed twice
    static_assert(NT == 1 || NST % NT == 0, "each MMA thread must meet every stage it uses on every turn of the K ring");
    int stage = 0, acc = 0, cur_u = -1;
    uint32_t fphase = 0, qfphase = 0, tephase0 = 1, tephase1 = 1;
    bool ok = true;
    for (int it = item_begin; it < item_end && ok; ++it) {
        if (FILTERED && p.redo && !p.redo[it]) continue;
        const int u = it / p.nchunk, j = it - u * p.nchunk;
        const int lo = j * p.chunk_keys, hi = min(p.N, lo + p.chunk_keys);
        const int nt = (hi - lo + TN - 1) / TN;
        if (nt <= 0) continue;
        if (u != cur_u) {
            if (cur_u >= 0) umma_commit(pp.qempty());     // Q may be replaced once these MMAs are done
            if (!(ok = mbar_wait_relaxed(pp.qfull(), qfphase, pp.abort_flag, p.err, p.wait_cycles))) break;
            qfphase ^= 1;
            cur_u = u;
        }
        for (int t = 0; t < nt; ++t) {
            const bool mine = NT == 1 || acc == which;
            if (mine) {
            if (!(ok = mbar_wait_relaxed(pp.full(stage), fphase, pp.abort_flag, p.err, p.wait_cycles))) break;
            const uint32_t tph = acc ? tephase1 : tephase0;
            const uint32_t kb = pp.sK + stage * Cfg::kStageBytes;
#pragma unroll
            for (int b = 0; b < MB; ++b) {
                if (!(ok = mbar_wait_relaxed(pp.tempty(acc, b), tph, pp.abort_flag, p.err, p.wait_cycles))) break;
                fence_after_sync();
                const uint32_t d_tmem = pp.tmem_base + (uint32_t)((acc * MB + b) * TN);
#pragma unroll
                for (int ks = 0; ks < KSTEPS; ++ks) {
                    const uint32_t a_addr = pp.sQ + (b * NSUB + (ks >> 2)) * Cfg::kSubBytes + (ks & 3) * 32;
                    const uint32_t b_addr = kb + (ks >> 2) * Cfg::kSubBytes + (ks & 3) * 32;
                    umma_bf16(d_tmem, smem_desc(a_addr), smem_desc(b_addr), idesc, ks > 0);
                }
                umma_commit(pp.tfull(acc, b));
            }
            if (!ok) break;
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

template <int D, int MB>
__global__ void __launch_bounds__(ScoreTcCfg<D, MB>::kThreads, 1)
    score_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const int q_box_rows,
                    const int k_box_rows, const ScoreTcParams p) {
    using Cfg = ScoreTcCfg<D, MB>;
    constexpr int TN = tc::kTileKeys;
    constexpr int NSL = Cfg::kSlices, SLW = TN / NSL, NCH = SLW / 32;     // slices, slice width, chunks per slice
    extern __shared__ unsigned char smem_raw[];
    if (p.redo_any && *p.redo_any == 0) return;       // repair launch with nothing to repair
    tc::stamp(p.clk, 0);
    tc::Pipe<Cfg> pp;
    tc::pipe_setup(pp, smem_raw, 16 / MB);
    float* comb = tc::pipe_scratch(pp, smem_raw);     // [2][4][128][2]
    const uint32_t tmem_base = pp.tmem_base;
    volatile int* abort_flag = pp.abort_flag;
    auto bar_tfull = [&](int a, int b) { return pp.tfull(a, b); };
    auto bar_tempty = [&](int a, int b) { return pp.tempty(a, b); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long total = p.total_items;
    const int item_begin = (int)(total * blockIdx.x / gridDim.x);
    const int item_end = (int)(total * (blockIdx.x + 1) / gridDim.x);

    if (warp == 0) {
        if (lane == 0) tc::producer_role<D, MB, true, false>(pp, &tmQ, &tmK, q_box_rows, k_box_rows, p, item_begin, item_end);
    } else if (warp == 1) {
        if (lane == 0) tc::mma_role<D, MB, true, 1>(pp, p, item_begin, item_end, 0);
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ epilogue
        // a warp may touch the 32 tensor-memory lanes given by its index modulo 4; any four
        // consecutive warps cover all 128 rows of a block
        const int g = (warp - 4) >> 2, quad = warp & 3;
        const int blk = MB == 2 ? (g >> 1) : 0;            // 128-row block of Q
        const int slice = MB == 2 ? (g & 1) : g;           // column slice of every tile
        const int lrow = quad * 32 + lane;
        const int row = blk * 128 + lrow;
        const int plim = row < p.R ? p.N - p.W + (row % p.W) : p.N - 1;
        const float scale = p.scale_log2;
        const int units_per_prompt = p.L * p.Hkv;
        int acc = 0, nflush = 0;
        uint32_t tfphase0 = 0, tfphase1 = 0;
        bool ok = true;
        for (int it = item_begin; it < item_end && ok; ++it) {
            if (p.redo) {
                if (!p.redo[it]) continue;
                if (warp == 4 && lane == 0) atomicAdd(p.repaired, 1);
            }
            const int u = it / p.nchunk, j = it - u * p.nchunk;
            const int lo = j * p.chunk_keys, hi = min(p.N, lo + p.chunk_keys);
            const int nt = (hi - lo + TN - 1) / TN;
            const int bprompt = u / units_per_prompt;
            const int2* pcs = p.pieces + (size_t)bprompt * p.P;
            int pi = p.chunk_first[(size_t)bprompt * p.cf_stride + j];
            const int pi_last = p.chunk_first[(size_t)bprompt * p.cf_stride + j + 1];
            int pend = pi < pi_last ? pcs[pi].y : 0x7fffffff;
            float m_ref = SHOTKV_NEG_INF, z = 0.f;
            const int plain_end = min(hi, p.N - p.W + 1);      // keys below this count for every window row

            // piece `pi` is complete for this thread's columns: merge the row's slices, write, move on
            auto flush = [&]() {
                // slot of warpgroup g' and local row r: comb[parity][g'][r][m, z]; a row's slices are the
                // NSL consecutive warpgroups starting at its leader (slice 0)
                float* slot = comb + (nflush & 1) * 1024 + (g - slice) * 256 + lrow * 2;
                if (slice != 0) {
                    slot[slice * 256] = m_ref;
                    slot[slice * 256 + 1] = z;
                }
                if (blk == 0) asm volatile("bar.sync 1, %0;" ::"n"(NSL * 128) : "memory");
                else asm volatile("bar.sync 2, %0;" ::"n"(NSL * 128) : "memory");
                if (slice == 0) {
                    float mm = m_ref;
#pragma unroll
                    for (int s = 1; s < NSL; ++s) mm = fmaxf(mm, slot[s * 256]);
                    const float mu = mm == SHOTKV_NEG_INF ? 0.f : mm;
                    float zz = z * ex2f(m_ref - mu);
#pragma unroll
                    for (int s = 1; s < NSL; ++s) zz += slot[s * 256 + 1] * ex2f(slot[s * 256] - mu);
                    const size_t o = ((size_t)u * p.P + pi) * p.Rpad + row;
                    const bool live = row < p.R;        // padding rows: their Q was never loaded
                    p.part_m[o] = live ? mm : 0.f;
                    p.part_z[o] = live ? zz : 0.f;
                }
                z = 0.f;
                ++nflush;
                ++pi;
                pend = pi < pi_last ? pcs[pi].y : 0x7fffffff;
            };

            // 32 columns of this thread's row, starting at key kc0
            auto chunk = [&](uint32_t (&r)[32], int kc0) {
                while (pend <= kc0) flush();
                const int lim = min(hi, plim + 1) - kc0;                 // columns of the chunk that count
                if (!__all_sync(0xffffffffu, lim >= 32)) tc::mask32(r, lim);   // end of the keys, or the causal window
                const float cm = tc::max32(r) * scale;
                if (cm > m_ref + 8.f) {                                   // also the first time (m_ref = -inf, z = 0)
                    z *= ex2f(m_ref - cm);
                    m_ref = cm;
                }
                const float neg = m_ref == SHOTKV_NEG_INF ? 0.f : -m_ref;
                if (pend >= kc0 + 32) {                                   // no piece ends inside the chunk
                    z += tc::expsum32(r, scale, neg);
                    return;
                }
                tc::exp32(r, scale, neg);
                const int pend2 = pi + 1 < pi_last ? pcs[pi + 1].y : 0x7fffffff;
                if (pend2 >= kc0 + 32) {                                  // exactly one boundary: one predicated pass
                    float lo_s, hi_s;
                    tc::split32(r, pend - kc0, lo_s, hi_s);
                    z += lo_s;
                    flush();
                    z = hi_s;
                } else {                                                  // several short pieces: general walk
                    int start = 0;
                    while (pend < kc0 + 32) {
                        const int e = pend - kc0;
                        z += tc::range32(r, start, e);
                        start = e;
                        flush();
                    }
                    z += tc::range32(r, start, 32);
                }
            };

            for (int t = 0; t < nt; ++t) {
                const uint32_t tph = acc ? tfphase1 : tfphase0;
                ok = lane == 0 ? tc::mbar_wait(bar_tfull(acc, blk), tph, abort_flag, p.err, p.wait_cycles) : true;   // one poller per warp
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                if (acc) tfphase1 ^= 1; else tfphase0 ^= 1;
                tc::fence_after_sync();
                const int kc0 = lo + t * TN + slice * SLW;
                const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)((acc * MB + blk) * TN + slice * SLW);
                while (pend <= kc0) flush();
                uint32_t r[32];
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    tc::tmem_ld32_sync(r, taddr + c * 32);
                    if (c == NCH - 1) {                                   // the last of this tile's accumulators are in registers
                        tc::fence_before_sync();
                        __syncwarp();
                        if (lane == 0) tc::mbar_arrive(bar_tempty(acc, blk));
                    }
                    // most chunks: every column counts for every row (it lies before the item's end and
                    // before the first window position) and no piece ends at or inside the chunk
                    if (kc0 + c * 32 + 32 <= min(pend, plain_end)) {
                        const float cm = tc::max32(r) * scale;
                        if (cm > m_ref + 8.f) {
                            z *= ex2f(m_ref - cm);
                            m_ref = cm;
                        }
                        z += tc::expsum32(r, scale, -m_ref);
                    } else {
                        chunk(r, kc0 + c * 32);
                    }
                }
                acc ^= 1;
            }
            if (!ok) break;
            while (pi < pi_last) flush();
        }
    }

    tc::fence_before_sync();
    __syncthreads();
    tc::stamp(p.clk, 1);
    if (warp == 0) {
        __syncwarp();
        tc::fence_after_sync();
        tc::tmem_dealloc(tmem_base, 512);
    }
}

// Self-test of the bounded waits, for the host to run on demand: one CTA, two warps, two mbarriers
// that nobody ever arrives on.  Warp 0 waits on the first the way the epilogue warps do (lane 0
// polls with mbar_wait, the result is shuffled to the warp) with the given limit; lane 0 of warp 1
// waits on the second the way the producer and MMA threads do (mbar_wait_relaxed) with four times
// the limit, so it must leave because warp 0 raised the abort flag, not because its own time ran
// out.  Tensor memory is allocated at the start and released at the end, as in the kernels' exit
// path after an abort.  report[0..3] = {warp 0's wait returned true, warp 1's wait returned true,
// abort flag at exit, cycles warp 1 waited (saturated at 2^31 - 1)}.  The error word is raised
// exactly as in a real give-up, so the next call on the context reports it.
__global__ void __launch_bounds__(64, 1) bounded_wait_selftest_kernel(long long limit, int* err, int* report) {
    __shared__ __align__(8) unsigned long long bars[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_word;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t bar0 = smem_u32(&bars[0]), bar1 = smem_u32(&bars[1]);
    volatile int* abort_flag = &abort_word;
    if (threadIdx.x == 0) {
        tc::mbar_init(bar0, 1);
        tc::mbar_init(bar1, 1);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        tc::tmem_alloc(smem_u32(&tmem_slot), 32);
        tc::tmem_relinquish();
    }
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    if (warp == 0) {
        bool ok = lane == 0 ? tc::mbar_wait(bar0, 0, abort_flag, err, limit) : true;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (lane == 0) report[0] = ok ? 1 : 0;
    } else if (lane == 0) {
        const long long t0 = clock64();
        const bool ok = tc::mbar_wait_relaxed(bar1, 0, abort_flag, err, 4 * limit);
        const long long dt = clock64() - t0;
        report[1] = ok ? 1 : 0;
        report[3] = dt > 0x7fffffffLL ? 0x7fffffff : (int)dt;
    }
    tc::fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0) report[2] = *abort_flag;
    if (warp == 0) {
        __syncwarp();
        tc::fence_after_sync();
        tc::tmem_dealloc(tmem_base, 32);
    }
}

}  // namespace shotkv
