// C ABI of the ShotKV hot path: argument validation, workspace carving and launch sequencing.
// Every arithmetic step runs in the kernels of this directory; there is no host fallback.
#include "../../include/shotkv.h"

#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <functional>
#include <new>
#include <vector>

#include "colsum_tc.cuh"
#include "common.cuh"
#include "decode.cuh"
#include "score_fast.cuh"
#include "score_stream.cuh"
#include "reductions.cuh"
#include "score_tc.cuh"
#include "select_compact.cuh"

using namespace shotkv;

namespace {

constexpr int kMaxChunks = 64;         // most chunks a unit's keys are split into for load balance
constexpr int kMaxShots = 8192;
constexpr int kStageSlots = 4;
constexpr size_t kStageSlotBytes = 1u << 20;
constexpr int kProfSlots = 64;
constexpr int kMaxGroups = 4;         // most groups the fused prefill call pipelines its units in
constexpr double kMinGroupKBytes = 256.0 * 1024 * 1024;   // least K a group of the automatic split holds
constexpr int kErrWords = 16;          // ints of host-mapped memory the kernels report through
constexpr int kBigSmem = 200 * 1024;   // dynamic shared memory the small kernels are allowed (set once per context)

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

// Tracing: every compute entry point of the ABI is an NVTX range named after it, so that a
// timeline tool shows which call enqueued which kernels.  NVTX is header-only and does nothing
// unless a tool is attached to the process.
struct TraceRange {
    explicit TraceRange(const char* name) { nvtxRangePushA(name); }
    ~TraceRange() { nvtxRangePop(); }
    TraceRange(const TraceRange&) = delete;
    TraceRange& operator=(const TraceRange&) = delete;
};

}  // namespace

struct shotkv_ctx {
    int device = 0;
    char err[512] = {0};
    // pinned staging ring for the small host tables (offsets, piece lists) that go to the device
    unsigned char* stage = nullptr;
    cudaEvent_t stage_done[kStageSlots] = {};
    int stage_next = 0;
    // optional stage timing: a ring of event sets, one per profiled call
    bool prof = false;
    cudaEvent_t prof_ev[kProfSlots][5] = {};
    int prof_marks[kProfSlots] = {};
    // the pipelined fused call records per group: scoring begin/end on the caller's stream, then
    // begin, reduce end, selection end, compaction end on the stream those steps ran on
    cudaEvent_t prof_gev[kProfSlots][kMaxGroups][6] = {};
    int prof_groups[kProfSlots] = {};
    int prof_calls = 0;
    // second stream of the fused prefill call: reduce + select + compact of one group of units run
    // there while the caller's stream scores the next group
    cudaStream_t aux = nullptr;
    cudaEvent_t ev_fork[kMaxGroups] = {};
    cudaEvent_t ev_join = nullptr;
    int pipeline_groups = 0;           // 0 = chosen from the sizes
    unsigned long long launches = 0;   // kernels launched through this context
    // error word that kernels with bounded waits raise; pinned host memory mapped into the device
    int* err_host = nullptr;
    int* err_dev = nullptr;
    int sm_count = 148;
    int scoring_mode = SHOTKV_SCORING_FAST;
    long long wait_cycles = tc::kWaitCycles;   // limit of every bounded device-side wait
    int32_t* static_offsets = nullptr;         // device address of the built-in boundary table (looked up on first use)
    void* encode_tiled = nullptr;              // cuTensorMapEncodeTiled, resolved at creation
};

namespace {

int fail(shotkv_ctx* ctx, int code, const char* fmt, ...) {
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
        va_end(ap);
    }
    return code;
}

#define CUDA_TRY(ctx, expr)                                                                     \
    do {                                                                                        \
        cudaError_t e__ = (expr);                                                               \
        if (e__ != cudaSuccess)                                                                 \
            return fail(ctx, SHOTKV_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e__)); \
    } while (0)

// After every kernel launch: count it and surface launch errors.
#define LAUNCH_CHECK(ctx)                    \
    do {                                     \
        (ctx)->launches += 1;                \
        CUDA_TRY(ctx, cudaGetLastError());   \
    } while (0)

// Records the next stage boundary of the current profiled call (no-op unless profiling is on).
void prof_begin(shotkv_ctx* ctx) {
    if (!ctx->prof) return;
    ctx->prof_calls += 1;
    ctx->prof_marks[(ctx->prof_calls - 1) % kProfSlots] = 0;
    ctx->prof_groups[(ctx->prof_calls - 1) % kProfSlots] = 0;
}
void prof_gmark(shotkv_ctx* ctx, int group, int mark, cudaStream_t stream) {
    if (!ctx->prof || ctx->prof_calls == 0) return;
    const int slot = (ctx->prof_calls - 1) % kProfSlots;
    if (group + 1 > ctx->prof_groups[slot]) ctx->prof_groups[slot] = group + 1;
    cudaEventRecord(ctx->prof_gev[slot][group][mark], stream);
}
void prof_mark(shotkv_ctx* ctx, cudaStream_t stream) {
    if (!ctx->prof || ctx->prof_calls == 0) return;
    const int slot = (ctx->prof_calls - 1) % kProfSlots;
    int& m = ctx->prof_marks[slot];
    if (m < 5) cudaEventRecord(ctx->prof_ev[slot][m++], stream);
}

int check_dims(const shotkv_dims* d, const char** why) {
    if (!d) { *why = "dims is NULL"; return SHOTKV_ERR_INVALID_ARG; }
    if (d->B < 1 || d->L < 1 || d->H < 1 || d->Hkv < 1 || d->N < 1 || d->W < 1 || d->S < 0) {
        *why = "B, L, H, Hkv, N, W must be >= 1 and S >= 0"; return SHOTKV_ERR_INVALID_ARG;
    }
    if (d->H % d->Hkv != 0) { *why = "H must be a multiple of Hkv"; return SHOTKV_ERR_INVALID_ARG; }
    if (d->W > d->N) { *why = "window W exceeds N"; return SHOTKV_ERR_INVALID_ARG; }
    if (d->d != 64 && d->d != 128) { *why = "head dimension must be 64 or 128"; return SHOTKV_ERR_UNSUPPORTED_SHAPE; }
    if ((long long)(d->H / d->Hkv) * d->W > 256) { *why = "G*W must be <= 256"; return SHOTKV_ERR_UNSUPPORTED_SHAPE; }
    if (d->S > kMaxShots) { *why = "S must be <= 8192"; return SHOTKV_ERR_UNSUPPORTED_SHAPE; }
    if ((long long)d->B * d->L * d->Hkv > 0x7fffffffLL / 256) { *why = "B*L*Hkv too large"; return SHOTKV_ERR_UNSUPPORTED_SHAPE; }
    return SHOTKV_OK;
}

int check_policy_prefill(const shotkv_policy* p, const char** why) {
    if (!p) { *why = "policy is NULL"; return SHOTKV_ERR_INVALID_ARG; }
    if (!(p->r_p > 0.f) || !std::isfinite(p->r_p)) { *why = "r_p must be a positive finite number"; return SHOTKV_ERR_INVALID_ARG; }
    if (p->select_mode != 0 && p->select_mode != 1) { *why = "select_mode must be 0 or 1"; return SHOTKV_ERR_INVALID_ARG; }
    return SHOTKV_OK;
}

int budget_of(const shotkv_dims* d, const shotkv_policy* p) {
    const double b = std::floor((double)p->r_p * (double)d->N);
    return b > (double)d->N ? d->N : (int)b;
}

// 0 ok, negative error, or the warning; *max_always = largest always-kept count over the prompts
int check_offsets(const shotkv_dims* d, const shotkv_policy* p, const int32_t* off, int* max_always, const char** why) {
    if (!off) { *why = "offsets_host is NULL"; return SHOTKV_ERR_INVALID_ARG; }
    int worst = 0;
    for (int b = 0; b < d->B; ++b) {
        const int32_t* o = off + (size_t)b * (d->S + 1);
        if (o[0] < 0) { *why = "off[0] < 0"; return SHOTKV_ERR_BAD_OFFSETS; }
        for (int i = 0; i < d->S; ++i)
            if (o[i + 1] <= o[i]) { *why = "offsets must be strictly increasing (no empty shot)"; return SHOTKV_ERR_BAD_OFFSETS; }
        if (o[d->S] > d->N - d->W) { *why = "off[S] > N - W: the window must lie after the last shot"; return SHOTKV_ERR_BAD_OFFSETS; }
        const int always = o[0] + (d->N - o[d->S]);
        if (always > worst) worst = always;
    }
    if (max_always) *max_always = worst;
    if (p && worst > budget_of(d, p)) return SHOTKV_WARN_BUDGET_BELOW_ALWAYS_KEPT;
    return SHOTKV_OK;
}

int rpad_of(const shotkv_dims* d) { return (d->H / d->Hkv) * d->W <= 128 ? 128 : 256; }
// Units shorter than this many tokens on average put several piece ends into every 32-column chunk
// of the scoring pass; the fused call then goes through per-token importances instead (two passes
// over K, cost independent of S).  Measured on 4 x 32 layers x 32,768 tokens: sentence-sized units
// (25 tokens on average) 5.7 ms single-pass against 6.8 ms two-pass, 16-token chunks 6.0 against
// 6.9, 12-token chunks 8.3 against 7.1, 8-token chunks 10.5 against 7.5.
// With 128 window rows or fewer a pass over K costs half the exponentials and the work of splitting
// chunks at piece ends weighs twice as much beside it: there the two-pass route wins from about 40
// tokens down (1 x 32 layers x 16,384 tokens, sentence-sized units: 0.71 ms against 0.95 ms single-pass).
constexpr int kTokenRouteBelowMeanLen = 16, kTokenRouteBelowMeanLenFewRows = 40;
bool token_route(const shotkv_dims* d) {
    const int below = rpad_of(d) > 128 ? kTokenRouteBelowMeanLen : kTokenRouteBelowMeanLenFewRows;
    return d->S > 0 && (long long)d->N < (long long)below * d->S;
}
// Pieces per prompt the workspace is sized for: shot boundaries plus chunk ends, or chunk ends alone
// when the shot-aware scoring pass is never run for these dims.
int pmax_of(const shotkv_dims* d) { return (token_route(d) ? 0 : d->S) + 2 + kMaxChunks + 1; }

struct PrefillWs {
    int* off;          // [B][S+1]
    int2* pieces;      // [B][Pmax]
    int* piece_seg;    // [B][Pmax]
    int* chunk_first;  // [B][kMaxChunks + 1]
    float* part_m;     // [U][Pmax][Rpad]
    float* part_z;
    float* item_m;     // [U * kMaxChunks][Rpad] per (work item, row): the reference its pieces share and the sum of their z
    float* item_z;
    float* row_m;      // [U][Rpad]
    float* row_invz;
    float* unit_shot;  // [U][S]
    float* imp;        // [U][N] per-token importances of the fused call's per-token route (absent otherwise)
    int* redo;         // [kMaxGroups + U * kMaxChunks] per group of units: one word "some item is marked", then one word per item the exact kernel must recompute
    size_t total;
};

PrefillWs carve(const shotkv_dims* d, void* base) {
    PrefillWs w{};
    const size_t U = (size_t)d->B * d->L * d->Hkv, P = pmax_of(d), R = rpad_of(d);
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o += align_up(bytes); return (unsigned char*)base + at; };
    w.off = (int*)take((size_t)d->B * (d->S + 1) * 4);
    w.pieces = (int2*)take((size_t)d->B * P * 8);
    w.piece_seg = (int*)take((size_t)d->B * P * 4);
    w.chunk_first = (int*)take((size_t)d->B * (kMaxChunks + 1) * 4);
    w.part_m = (float*)take(U * P * R * 4);
    w.part_z = (float*)take(U * P * R * 4);
    w.item_m = (float*)take(U * kMaxChunks * R * 4);
    w.item_z = (float*)take(U * kMaxChunks * R * 4);
    w.row_m = (float*)take(U * R * 4);
    w.row_invz = (float*)take(U * R * 4);
    w.unit_shot = (float*)take(U * (size_t)(d->S > 0 ? d->S : 1) * 4);
    w.imp = (float*)take(token_route(d) ? U * (size_t)d->N * 4 : 0);
    w.redo = (int*)take((U * kMaxChunks + kMaxGroups) * 4);
    w.total = o;
    return w;
}

// Copies `bytes` of host data to `dst` on `stream` through the context's pinned ring, so the
// caller's buffer may be reused at once and the host does not wait for the stream.
int upload_small(shotkv_ctx* ctx, void* dst, const void* src, size_t bytes, cudaStream_t stream) {
    // one ring slot at a time; a table larger than a slot goes in several copies.  The host waits
    // only for the copy that last used the slot it is about to refill, never for the stream.
    for (size_t done = 0; done < bytes;) {
        const size_t n = bytes - done < kStageSlotBytes ? bytes - done : kStageSlotBytes;
        const int slot = ctx->stage_next;
        ctx->stage_next = (slot + 1) % kStageSlots;
        CUDA_TRY(ctx, cudaEventSynchronize(ctx->stage_done[slot]));
        unsigned char* s = ctx->stage + (size_t)slot * kStageSlotBytes;
        memcpy(s, (const unsigned char*)src + done, n);
        CUDA_TRY(ctx, cudaMemcpyAsync((unsigned char*)dst + done, s, n, cudaMemcpyHostToDevice, stream));
        CUDA_TRY(ctx, cudaEventRecord(ctx->stage_done[slot], stream));
        done += n;
    }
    return SHOTKV_OK;
}

// Work partition of the scoring pass.  Every unit's keys are cut into `nchunk` chunks of
// `chunk_keys` keys (whole 128-key tiles); an item is one (unit, chunk) and the persistent CTAs
// take equal runs of consecutive items.  The split that minimises the busiest CTA's tile count
// wins; each extra chunk costs one more piece per unit, so ties go to fewer chunks.
struct ChunkPlan { int nchunk, chunk_keys; };
ChunkPlan plan_chunks(const shotkv_dims* d, int sm_count) {
    const long long U = (long long)d->B * d->L * d->Hkv;
    const int tiles = (d->N + 127) / 128;
    ChunkPlan best{1, tiles * 128};
    long long best_cost = -1;
    for (int want = 1; want <= kMaxChunks && want <= tiles; ++want) {
        const int ct = (tiles + want - 1) / want;             // tiles per chunk
        const int nchunk = (tiles + ct - 1) / ct;
        const long long items = U * nchunk;
        const long long ctas = items < sm_count ? items : sm_count;
        const long long per_cta = (items + ctas - 1) / ctas;
        const long long cost = per_cta * (ct * 16 + 3);       // a tile plus a small per-item overhead, in 1/16 tiles
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            best = ChunkPlan{nchunk, ct * 128};
        }
    }
    return best;
}

// Cuts [0, N) of every prompt into pieces at the chunk ends and, when offsets are given, at the
// segment boundaries (segment 0 = before the first shot, i+1 = shot i, S+1 = the question).
// piece_seg records each piece's segment (S+2 marks list padding); chunk_first[b][j] is the index
// of the first piece of chunk j.  Returns pieces per prompt (the same for all after padding).
int build_pieces(const shotkv_dims* d, const int32_t* off, const ChunkPlan& plan, std::vector<int2>& pieces,
                 std::vector<int>& seg, std::vector<int>& chunk_first) {
    std::vector<std::vector<int2>> pp(d->B);
    std::vector<std::vector<int>> ss(d->B);
    chunk_first.assign((size_t)d->B * (kMaxChunks + 1), 0);
    size_t P = 0;
    for (int b = 0; b < d->B; ++b) {
        int* cf = chunk_first.data() + (size_t)b * (kMaxChunks + 1);
        int next_chunk = 0;
        auto add_range = [&](int lo, int hi, int s) {
            int x = lo;
            while (x < hi) {
                const int j = x / plan.chunk_keys;
                const int cend = (j + 1) * plan.chunk_keys;
                const int y = cend < hi ? cend : hi;
                while (next_chunk <= j) cf[next_chunk++] = (int)pp[b].size();
                pp[b].push_back(make_int2(x, y));
                ss[b].push_back(s);
                x = y;
            }
        };
        if (off) {
            const int32_t* o = off + (size_t)b * (d->S + 1);
            add_range(0, o[0], 0);
            for (int i = 0; i < d->S; ++i) add_range(o[i], o[i + 1], i + 1);
            add_range(o[d->S], d->N, d->S + 1);
        } else {
            add_range(0, d->N, 0);
        }
        while (next_chunk <= plan.nchunk) cf[next_chunk++] = (int)pp[b].size();
        if (pp[b].size() > P) P = pp[b].size();
    }
    if (P == 0) P = 1;
    pieces.assign((size_t)d->B * P, make_int2(d->N, d->N));
    seg.assign((size_t)d->B * P, d->S + 2);
    for (int b = 0; b < d->B; ++b)
        for (size_t i = 0; i < pp[b].size(); ++i) {
            pieces[(size_t)b * P + i] = pp[b][i];
            seg[(size_t)b * P + i] = ss[b][i];
        }
    return (int)P;
}

int set_device(shotkv_ctx* ctx) {
    if (!ctx) return SHOTKV_ERR_INVALID_ARG;
    CUDA_TRY(ctx, cudaSetDevice(ctx->device));
    if (ctx->err_host && *(volatile int*)ctx->err_host) {
        *(volatile int*)ctx->err_host = 0;
        return fail(ctx, SHOTKV_ERR_TIMEOUT, "an earlier scoring kernel gave up a bounded wait; its outputs are invalid");
    }
    return SHOTKV_OK;
}

// ---- tensor-core scoring: tensor maps and launch ----------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Resolved once per context, at creation (no process-wide state).
void* resolve_encode_tiled() {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
        return p;
    return nullptr;
}

template <int D, int MB>
int launch_score_tc_t(shotkv_ctx* ctx, const CUtensorMap& tmQ, const CUtensorMap& tmK, int qbox, int kbox,
                      const ScoreTcParams& sp, cudaStream_t stream) {
    constexpr int smem = ScoreTcCfg<D, MB>::kSmemBytes;
    int grid = sp.total_items < ctx->sm_count ? sp.total_items : ctx->sm_count;
    if (grid < 1) grid = 1;
    score_tc_kernel<D, MB><<<grid, ScoreTcCfg<D, MB>::kThreads, smem, stream>>>(tmQ, tmK, qbox, kbox, sp);
    LAUNCH_CHECK(ctx);
    return SHOTKV_OK;
}

// Column pairs, of every 16, whose exponentials run on the FMA pipe instead of the special-function unit.
constexpr int kPolyEvery = 5;

template <int D>
int launch_score_fast_t(shotkv_ctx* ctx, const CUtensorMap& tmQ, const CUtensorMap& tmK, int qbox, int kbox,
                        const ScoreTcParams& sp, cudaStream_t stream) {
    constexpr int smem = ScoreFastCfg<D>::kSmemBytes;
    int grid = sp.total_items < ctx->sm_count ? sp.total_items : ctx->sm_count;
    if (grid < 1) grid = 1;
    score_fast_kernel<D, kPolyEvery><<<grid, ScoreFastCfg<D>::kThreads, smem, stream>>>(tmQ, tmK, qbox, kbox, sp);
    LAUNCH_CHECK(ctx);
    return SHOTKV_OK;
}

template <int D>
int launch_score_stream_t(shotkv_ctx* ctx, const CUtensorMap& tmQ, const CUtensorMap& tmK, int qbox, int kbox,
                          const ScoreTcParams& sp, cudaStream_t stream) {
    using Cfg = ScoreStreamCfg<D>;
    int grid = sp.total_items < ctx->sm_count ? sp.total_items : ctx->sm_count;
    if (grid < 1) grid = 1;
    score_stream_kernel<D, kPolyEvery><<<grid, Cfg::kThreads, Cfg::kSmemBytes, stream>>>(tmQ, tmK, qbox, kbox, sp);
    LAUNCH_CHECK(ctx);
    return SHOTKV_OK;
}

// Tensor maps of Q (2-D: d x rows) and K (3-D: d x N x units), 64-element boxes with 128-byte swizzle, and the
// parameters every tensor-core pass shares.
struct TcSetup {
    CUtensorMap tmQ, tmK;
    int qbox, kbox;
    ScoreTcParams sp;
};
int tc_setup(shotkv_ctx* ctx, const shotkv_dims* d, const shotkv_bf16* Q, const shotkv_bf16* K, const PrefillWs& w, int P,
             const ChunkPlan& plan, TcSetup& t) {
    EncodeTiledFn enc = (EncodeTiledFn)ctx->encode_tiled;
    if (!enc) return fail(ctx, SHOTKV_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
    if (((uintptr_t)Q | (uintptr_t)K) & 15) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "Qwin and K must be 16-byte aligned");
    const long long U = (long long)d->B * d->L * d->Hkv;
    const int R = (d->H / d->Hkv) * d->W;
    const long long qrows = U * R;
    t.qbox = qrows < 128 ? (int)qrows : 128;
    t.kbox = d->N < 128 ? d->N : 128;
    {
        cuuint64_t dims[2] = {(cuuint64_t)d->d, (cuuint64_t)qrows};
        cuuint64_t strides[1] = {(cuuint64_t)d->d * 2};
        cuuint32_t box[2] = {64, (cuuint32_t)t.qbox}, es[2] = {1, 1};
        CUresult r = enc(&t.tmQ, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void*)Q, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail(ctx, SHOTKV_ERR_CUDA, "cuTensorMapEncodeTiled(Qwin) failed with %d", (int)r);
    }
    {
        cuuint64_t dims[3] = {(cuuint64_t)d->d, (cuuint64_t)d->N, (cuuint64_t)U};
        cuuint64_t strides[2] = {(cuuint64_t)d->d * 2, (cuuint64_t)d->N * d->d * 2};
        cuuint32_t box[3] = {64, (cuuint32_t)t.kbox, 1}, es[3] = {1, 1, 1};
        CUresult r = enc(&t.tmK, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, (void*)K, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail(ctx, SHOTKV_ERR_CUDA, "cuTensorMapEncodeTiled(K) failed with %d", (int)r);
    }
    ScoreTcParams& sp = t.sp;
    sp = ScoreTcParams{};
    sp.pieces = w.pieces;
    sp.chunk_first = w.chunk_first;
    sp.cf_stride = kMaxChunks + 1;
    sp.P = P;
    sp.nchunk = plan.nchunk;
    sp.chunk_keys = plan.chunk_keys;
    sp.L = d->L; sp.Hkv = d->Hkv; sp.N = d->N; sp.W = d->W; sp.R = R; sp.Rpad = rpad_of(d);
    if (U * plan.nchunk > 0x7fffffffLL) return fail(ctx, SHOTKV_ERR_UNSUPPORTED_SHAPE, "too many work items");
    sp.total_items = (int)(U * plan.nchunk);
    sp.scale_log2 = kLog2e / sqrtf((float)d->d);
    sp.part_m = w.part_m; sp.part_z = w.part_z;
    sp.item_m = w.item_m; sp.item_z = w.item_z;
    sp.err = ctx->err_dev;
    sp.wait_cycles = ctx->wait_cycles;
    sp.repaired = ctx->err_dev + 1;
    return SHOTKV_OK;
}

template <int D, int MB>
int launch_colsum_tc_t(shotkv_ctx* ctx, const TcSetup& t, const ColsumTcParams& cp, cudaStream_t stream) {
    constexpr int smem = ColsumTcCfg<D, MB>::kSmemBytes;
    int grid = cp.base.total_items < ctx->sm_count ? cp.base.total_items : ctx->sm_count;
    if (grid < 1) grid = 1;
    colsum_tc_kernel<D, MB, kPolyEvery><<<grid, ColsumTcCfg<D, MB>::kThreads, smem, stream>>>(t.tmQ, t.tmK, t.qbox, t.kbox, cp);
    LAUNCH_CHECK(ctx);
    return SHOTKV_OK;
}

// Second pass of the per-token path: token_importance from the row statistics in the workspace.
int launch_colsum_tc(shotkv_ctx* ctx, const shotkv_dims* d, const shotkv_bf16* Q, const shotkv_bf16* K, const PrefillWs& w,
                     float* imp, cudaStream_t stream) {
    TcSetup t;
    const ChunkPlan plan = plan_chunks(d, ctx->sm_count);
    int rc = tc_setup(ctx, d, Q, K, w, 0, plan, t);
    if (rc) return rc;
    ColsumTcParams cp{};
    cp.base = t.sp;
    cp.row_m = w.row_m; cp.row_invz = w.row_invz; cp.imp = imp;
    const bool big = t.sp.Rpad == 256;
    if (d->d == 128) return big ? launch_colsum_tc_t<128, 2>(ctx, t, cp, stream) : launch_colsum_tc_t<128, 1>(ctx, t, cp, stream);
    return big ? launch_colsum_tc_t<64, 2>(ctx, t, cp, stream) : launch_colsum_tc_t<64, 1>(ctx, t, cp, stream);
}

int launch_score_tc(shotkv_ctx* ctx, const shotkv_dims* d, const shotkv_bf16* Q, const shotkv_bf16* K, const PrefillWs& w,
                    int P, const ChunkPlan& plan, cudaStream_t stream) {
    TcSetup t;
    int rc0 = tc_setup(ctx, d, Q, K, w, P, plan, t);
    if (rc0) return rc0;
    const CUtensorMap& tmQ = t.tmQ;
    const CUtensorMap& tmK = t.tmK;
    const int qbox = t.qbox, kbox = t.kbox;
    ScoreTcParams& sp = t.sp;
    const bool big = sp.Rpad == 256;
    int rc = SHOTKV_OK;
    sp.clk = (long long*)(ctx->err_dev + 8);        // the first launch below stamps its clocks; a repair launch after it does not
    if (ctx->scoring_mode == SHOTKV_SCORING_FAST) {
        // fast kernel first; it marks the items whose sums left its range, and the exact kernel
        // below then redoes exactly those (returning at once when there is none)
        sp.redo_any = w.redo;
        sp.redo = w.redo + 1;
        CUDA_TRY(ctx, cudaMemsetAsync(w.redo, 0, ((size_t)sp.total_items + 1) * 4, stream));
        if (d->d == 128) rc = big ? launch_score_stream_t<128>(ctx, tmQ, tmK, qbox, kbox, sp, stream) : launch_score_fast_t<128>(ctx, tmQ, tmK, qbox, kbox, sp, stream);
        else rc = big ? launch_score_stream_t<64>(ctx, tmQ, tmK, qbox, kbox, sp, stream) : launch_score_fast_t<64>(ctx, tmQ, tmK, qbox, kbox, sp, stream);
        if (rc) return rc;
        sp.clk = nullptr;
    }
    if (d->d == 128) return big ? launch_score_tc_t<128, 2>(ctx, tmQ, tmK, qbox, kbox, sp, stream) : launch_score_tc_t<128, 1>(ctx, tmQ, tmK, qbox, kbox, sp, stream);
    return big ? launch_score_tc_t<64, 2>(ctx, tmQ, tmK, qbox, kbox, sp, stream) : launch_score_tc_t<64, 1>(ctx, tmQ, tmK, qbox, kbox, sp, stream);
}

int check_ws(shotkv_ctx* ctx, const shotkv_dims* d, void* ws, size_t ws_bytes) {
    if (!ws) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "workspace is NULL");
    if ((uintptr_t)ws % 256) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
    const size_t need = shotkv_workspace_bytes(d);
    if (ws_bytes < need) return fail(ctx, SHOTKV_ERR_WORKSPACE_TOO_SMALL, "workspace has %zu bytes, %zu needed", ws_bytes, need);
    return SHOTKV_OK;
}

// Builds the piece lists of every prompt for `plan` and uploads them with the chunk index.
int prepare_pieces(shotkv_ctx* ctx, const shotkv_dims* d, const int32_t* off_host, const ChunkPlan& plan, const PrefillWs& w,
                   int* P_out, cudaStream_t stream) {
    std::vector<int2> pieces;
    std::vector<int> seg, chunk_first;
    const int P = build_pieces(d, off_host, plan, pieces, seg, chunk_first);
    if (P > pmax_of(d)) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "internal: piece count %d exceeds bound %d", P, pmax_of(d));
    int rc = upload_small(ctx, w.pieces, pieces.data(), pieces.size() * sizeof(int2), stream);
    if (rc) return rc;
    rc = upload_small(ctx, w.piece_seg, seg.data(), seg.size() * sizeof(int), stream);
    if (rc) return rc;
    rc = upload_small(ctx, w.chunk_first, chunk_first.data(), chunk_first.size() * sizeof(int), stream);
    if (rc) return rc;
    *P_out = P;
    return SHOTKV_OK;
}

// What the scoring pass just left in `w`, as the reductions read it.
PartialView partial_view(const shotkv_ctx* ctx, const shotkv_dims* d, const PrefillWs& w, int P, const ChunkPlan& plan) {
    PartialView v{};
    v.part_m = w.part_m; v.part_z = w.part_z; v.item_m = w.item_m; v.item_z = w.item_z;
    v.all_exact = ctx->scoring_mode == SHOTKV_SCORING_EXACT ? 1 : 0;
    v.redo = v.all_exact ? nullptr : w.redo + 1;
    v.chunk_first = w.chunk_first;
    v.cf_stride = kMaxChunks + 1;
    v.nchunk = plan.nchunk;
    v.P = P;
    v.Rpad = rpad_of(d);
    return v;
}

// STATS pass over `pieces` followed by the per-row reduction; leaves part_m/part_z (and for the
// token path row_m/row_invz) in the workspace.
int run_stats(shotkv_ctx* ctx, const shotkv_dims* d, const shotkv_bf16* Q, const shotkv_bf16* K, const PrefillWs& w,
              const int32_t* off_host, bool need_rows, int* P_out, cudaStream_t stream) {
    const ChunkPlan plan = plan_chunks(d, ctx->sm_count);
    int P = 0;
    int rc = prepare_pieces(ctx, d, off_host, plan, w, &P, stream);
    if (rc) return rc;
    const int U = d->B * d->L * d->Hkv;
    prof_mark(ctx, stream);
    rc = launch_score_tc(ctx, d, Q, K, w, P, plan, stream);
    if (rc) return rc;
    prof_mark(ctx, stream);
    if (need_rows) {
        row_stats_kernel<<<U, 256, 0, stream>>>(partial_view(ctx, d, w, P, plan), d->L * d->Hkv, (d->H / d->Hkv) * d->W, w.row_m, w.row_invz);
        LAUNCH_CHECK(ctx);
    }
    *P_out = P;
    return SHOTKV_OK;
}

// ---- the fused call's pipeline over groups of units ---------------------------------------------
// Units (b, l) are independent, so the fused call may cut them into groups -- whole prompts, or
// runs of layers when there is one prompt -- and reduce, select and compact one group on a second
// stream while the caller's stream works on the next.  With host buffers that hides the write-back
// of one group's Kc/Vc behind the upload of the next group's K (the bus carries both directions at
// once).  With device buffers it measured no gain (the scoring pass slows by what the overlapped
// compaction takes: both draw on the same power budget and SMs) and a loss on small inputs, so
// there the automatic choice is one group.
struct GroupSplit {
    int n;          // groups
    int per;        // prompts (or layers, when by_layer) in every group but possibly the last
    bool by_layer;  // one prompt, cut along its layers
};
GroupSplit plan_groups(const shotkv_ctx* ctx, const shotkv_dims* d, bool host_staged) {
    GroupSplit g{1, 0, d->B == 1};
    const int count = g.by_layer ? d->L : d->B;
    int want = ctx->pipeline_groups;
    if (want <= 0) {
        // automatic: for host buffers one group per kMinGroupKBytes of K; otherwise one group
        const double k_bytes = (double)d->B * d->L * d->Hkv * d->N * d->d * 2.0;
        want = host_staged ? (int)(k_bytes / kMinGroupKBytes) : 1;
    }
    if (want > kMaxGroups) want = kMaxGroups;
    if (want > count) want = count;
    if (want < 1) want = 1;
    g.per = (count + want - 1) / want;
    g.n = (count + g.per - 1) / g.per;
    return g;
}
// One group's share of the call: its dims, and the offsets of its first prompt, first (b, l) pair and first unit.
struct GroupView {
    shotkv_dims d;
    size_t b0, bl0, u0;
};
GroupView group_view(const shotkv_dims* d, const GroupSplit& gs, int g) {
    GroupView v{};
    v.d = *d;
    const int count = gs.by_layer ? d->L : d->B;
    const int first = g * gs.per;
    const int n = first + gs.per <= count ? gs.per : count - first;
    if (gs.by_layer) { v.d.L = n; v.b0 = 0; v.bl0 = (size_t)first; }
    else { v.d.B = n; v.b0 = (size_t)first; v.bl0 = (size_t)first * d->L; }
    v.u0 = v.bl0 * d->Hkv;
    return v;
}
// The group's slices of the workspace arrays (P = pieces per prompt as uploaded).
PrefillWs group_ws(const PrefillWs& w, const shotkv_dims* d, const GroupView& v, int g, int P) {
    PrefillWs x = w;
    const size_t R = rpad_of(d);
    x.off = w.off + v.b0 * (d->S + 1);
    x.pieces = w.pieces + v.b0 * P;
    x.piece_seg = w.piece_seg + v.b0 * P;
    x.chunk_first = w.chunk_first + v.b0 * (kMaxChunks + 1);
    x.part_m = w.part_m + v.u0 * P * R;
    x.part_z = w.part_z + v.u0 * P * R;
    x.item_m = w.item_m + v.u0 * kMaxChunks * R;
    x.item_z = w.item_z + v.u0 * kMaxChunks * R;
    x.row_m = w.row_m + v.u0 * R;
    x.row_invz = w.row_invz + v.u0 * R;
    x.unit_shot = w.unit_shot + v.u0 * (size_t)(d->S > 0 ? d->S : 1);
    x.redo = w.redo + g + v.u0 * kMaxChunks;
    return x;
}

int run_select(shotkv_ctx* ctx, const shotkv_dims* d, const shotkv_policy* p, const PrefillWs& w, float* shot_scores,
               uint8_t* keep, int32_t* kept_idx, int32_t* kept_count, int32_t Mcap, cudaStream_t stream) {
    const size_t smem = (size_t)d->S * 16 + (kSelectThreads + 1) * 4 + 16;
    select_shots_kernel<<<d->B * d->L, kSelectThreads, smem, stream>>>(shot_scores, w.off, d->L, d->N, d->S, budget_of(d, p),
                                                                     p->select_mode, Mcap, keep, kept_idx, kept_count);
    LAUNCH_CHECK(ctx);
    return SHOTKV_OK;
}

int run_compact(shotkv_ctx* ctx, const shotkv_dims* d, const shotkv_bf16* K, const shotkv_bf16* V, const int32_t* kept_idx,
                const int32_t* kept_count, int32_t Mcap, shotkv_bf16* Kc, shotkv_bf16* Vc, cudaStream_t stream) {
    const int rows_per_cta = d->d == 128 ? 64 : 128;
    int gx = (Mcap + rows_per_cta - 1) / rows_per_cta;
    if (gx < 1) gx = 1;
    dim3 grid(gx, d->Hkv, d->B * d->L);
    if (grid.z > 65535) return fail(ctx, SHOTKV_ERR_UNSUPPORTED_SHAPE, "B*L must be <= 65535");
    if (d->d == 128)
        compact_kv_kernel<128><<<grid, 256, 0, stream>>>((const uint4*)K, (const uint4*)V, kept_idx, kept_count, d->Hkv, d->N, Mcap, (uint4*)Kc, (uint4*)Vc);
    else
        compact_kv_kernel<64><<<grid, 256, 0, stream>>>((const uint4*)K, (const uint4*)V, kept_idx, kept_count, d->Hkv, d->N, Mcap, (uint4*)Kc, (uint4*)Vc);
    LAUNCH_CHECK(ctx);
    return SHOTKV_OK;
}

// Dynamic shared-memory limits of every kernel that may need more than the 48 KB default.  A
// function attribute belongs to the device's context, so it is set once when a shotkv_ctx is
// created on that device, never on a launch path.
template <int D, int MB>
cudaError_t set_tc_attributes() {
    cudaError_t e = cudaFuncSetAttribute(score_tc_kernel<D, MB>, cudaFuncAttributeMaxDynamicSharedMemorySize, ScoreTcCfg<D, MB>::kSmemBytes);
    // the first scoring launch: one 128-row block of Q -> score_fast_kernel, two -> score_stream_kernel
    if (e == cudaSuccess && MB == 1)
        e = cudaFuncSetAttribute(score_fast_kernel<D, kPolyEvery>, cudaFuncAttributeMaxDynamicSharedMemorySize, ScoreFastCfg<D>::kSmemBytes);
    if (e == cudaSuccess && MB == 2)
        e = cudaFuncSetAttribute(score_stream_kernel<D, kPolyEvery>, cudaFuncAttributeMaxDynamicSharedMemorySize, ScoreStreamCfg<D>::kSmemBytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(colsum_tc_kernel<D, MB, kPolyEvery>, cudaFuncAttributeMaxDynamicSharedMemorySize, ColsumTcCfg<D, MB>::kSmemBytes);
    return e;
}
cudaError_t set_kernel_attributes() {
    cudaError_t e = set_tc_attributes<128, 1>();
    if (e == cudaSuccess) e = set_tc_attributes<128, 2>();
    if (e == cudaSuccess) e = set_tc_attributes<64, 1>();
    if (e == cudaSuccess) e = set_tc_attributes<64, 2>();
    const void* small[] = {(const void*)select_shots_kernel, (const void*)shot_mass_kernel<128>, (const void*)shot_mass_kernel<256>,
                           (const void*)decode_score_kernel<128>, (const void*)decode_score_kernel<64>,
                           (const void*)decode_attend_kernel<128>, (const void*)decode_attend_kernel<64>,
                           (const void*)decode_rank_kernel};
    for (const void* f : small)
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, kBigSmem);
    // the fused decode step wants three CTAs of ~74 KB each on an SM: ask for the largest shared-memory carve-out
    const void* wide[] = {(const void*)decode_attend_kernel<128>, (const void*)decode_attend_kernel<64>};
    for (const void* f : wide)
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    return e;
}

}  // namespace

// ------------------------------------------------------------------------------------------------
extern "C" {

const char* shotkv_version(void) { return "shotkv-b200 0.1"; }

int shotkv_create(shotkv_ctx** out, int device) {
    if (!out) return SHOTKV_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return SHOTKV_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return SHOTKV_ERR_CUDA;
    if (prop.major != 10) return SHOTKV_ERR_CUDA;   // built for sm_100a only
    if (cudaSetDevice(device) != cudaSuccess) return SHOTKV_ERR_CUDA;
    shotkv_ctx* ctx = new (std::nothrow) shotkv_ctx;
    if (!ctx) return SHOTKV_ERR_INVALID_ARG;
    ctx->device = device;
    if (cudaMallocHost((void**)&ctx->stage, kStageSlots * kStageSlotBytes) != cudaSuccess) {
        delete ctx;
        return SHOTKV_ERR_CUDA;
    }
    for (int i = 0; i < kStageSlots; ++i)
        if (cudaEventCreateWithFlags(&ctx->stage_done[i], cudaEventDisableTiming) != cudaSuccess) {
            cudaFreeHost(ctx->stage);
            delete ctx;
            return SHOTKV_ERR_CUDA;
        }
    if (cudaHostAlloc((void**)&ctx->err_host, kErrWords * sizeof(int), cudaHostAllocMapped) != cudaSuccess ||
        cudaHostGetDevicePointer((void**)&ctx->err_dev, ctx->err_host, 0) != cudaSuccess) {
        shotkv_destroy(ctx);
        return SHOTKV_ERR_CUDA;
    }
    bool ok = cudaStreamCreateWithFlags(&ctx->aux, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < kMaxGroups; ++i) ok = cudaEventCreateWithFlags(&ctx->ev_fork[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
        shotkv_destroy(ctx);
        return SHOTKV_ERR_CUDA;
    }
    for (int i = 0; i < kErrWords; ++i) ctx->err_host[i] = 0;   // word 0: a bounded wait gave up; word 1: work items the
                                                                 // exact scoring kernel recomputed; words 2-5: self-test report;
                                                                 // words 8-15: four 64-bit clock stamps of the last scoring launch
    ctx->sm_count = prop.multiProcessorCount;
    ctx->encode_tiled = resolve_encode_tiled();
    if (set_kernel_attributes() != cudaSuccess) {
        shotkv_destroy(ctx);
        return SHOTKV_ERR_CUDA;
    }
    *out = ctx;
    return SHOTKV_OK;
}

void shotkv_destroy(shotkv_ctx* ctx) {
    if (!ctx) return;
    cudaSetDevice(ctx->device);
    for (int i = 0; i < kStageSlots; ++i)
        if (ctx->stage_done[i]) {
            cudaEventSynchronize(ctx->stage_done[i]);
            cudaEventDestroy(ctx->stage_done[i]);
        }
    if (ctx->aux) {
        cudaStreamSynchronize(ctx->aux);
        cudaStreamDestroy(ctx->aux);
    }
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    for (int i = 0; i < kMaxGroups; ++i)
        if (ctx->ev_fork[i]) cudaEventDestroy(ctx->ev_fork[i]);
    if (ctx->stage) cudaFreeHost(ctx->stage);
    if (ctx->err_host) cudaFreeHost(ctx->err_host);
    for (int i = 0; i < kProfSlots; ++i) {
        for (int j = 0; j < 5; ++j)
            if (ctx->prof_ev[i][j]) cudaEventDestroy(ctx->prof_ev[i][j]);
        for (int g = 0; g < kMaxGroups; ++g)
            for (int j = 0; j < 6; ++j)
                if (ctx->prof_gev[i][g][j]) cudaEventDestroy(ctx->prof_gev[i][g][j]);
    }
    delete ctx;
}

const char* shotkv_last_error(const shotkv_ctx* ctx) { return ctx ? ctx->err : "context is NULL"; }

int32_t shotkv_budget_tokens(const shotkv_dims* dims, const shotkv_policy* policy) {
    const char* why = "";
    if (check_dims(dims, &why) || check_policy_prefill(policy, &why)) return SHOTKV_ERR_INVALID_ARG;
    return budget_of(dims, policy);
}

int32_t shotkv_kept_capacity(const shotkv_dims* dims, const shotkv_policy* policy, const int32_t* offsets_host) {
    const char* why = "";
    int rc = check_dims(dims, &why);
    if (rc) return rc;
    rc = check_policy_prefill(policy, &why);
    if (rc) return rc;
    int worst = 0;
    rc = check_offsets(dims, policy, offsets_host, &worst, &why);
    if (rc < 0) return rc;
    const int b = budget_of(dims, policy);
    return b > worst ? b : worst;
}

int shotkv_validate(const shotkv_dims* dims, const shotkv_policy* policy, const int32_t* offsets_host) {
    const char* why = "";
    int rc = check_dims(dims, &why);
    if (rc) return rc;
    if (policy) {
        rc = check_policy_prefill(policy, &why);
        if (rc) return rc;
    }
    if (offsets_host) return check_offsets(dims, policy, offsets_host, nullptr, &why);
    return SHOTKV_OK;
}

size_t shotkv_workspace_bytes(const shotkv_dims* dims) {
    const char* why = "";
    if (check_dims(dims, &why)) return 0;
    return carve(dims, nullptr).total;
}

int shotkv_prefill_score(shotkv_ctx* ctx, const shotkv_dims* dims, const shotkv_bf16* Qwin, const shotkv_bf16* K,
                         float* token_importance, void* ws, size_t ws_bytes, void* stream_) {
    TraceRange trace_("shotkv_prefill_score");
    int rc = set_device(ctx);
    if (rc) return rc;
    const char* why = "";
    if ((rc = check_dims(dims, &why))) return fail(ctx, rc, "%s", why);
    if (!Qwin || !K || !token_importance) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "Qwin, K and token_importance must not be NULL");
    if ((rc = check_ws(ctx, dims, ws, ws_bytes))) return rc;
    cudaStream_t stream = (cudaStream_t)stream_;
    const PrefillWs w = carve(dims, ws);
    int P = 0;
    if ((rc = run_stats(ctx, dims, Qwin, K, w, nullptr, true, &P, stream))) return rc;
    return launch_colsum_tc(ctx, dims, Qwin, K, w, token_importance, stream);
}

int shotkv_select_shots(shotkv_ctx* ctx, const shotkv_dims* dims, const shotkv_policy* policy,
                        const float* token_importance, const int32_t* offsets_host, float* shot_scores, uint8_t* keep,
                        int32_t* kept_idx, int32_t* kept_count, int32_t Mcap, void* ws, size_t ws_bytes, void* stream_) {
    TraceRange trace_("shotkv_select_shots");
    int rc = set_device(ctx);
    if (rc) return rc;
    const char* why = "";
    if ((rc = check_dims(dims, &why))) return fail(ctx, rc, "%s", why);
    if ((rc = check_policy_prefill(policy, &why))) return fail(ctx, rc, "%s", why);
    int worst = 0;
    const int orc = check_offsets(dims, policy, offsets_host, &worst, &why);
    if (orc < 0) return fail(ctx, orc, "%s", why);
    if (!shot_scores || !keep || !kept_idx || !kept_count) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "output pointers must not be NULL");
    const int need = budget_of(dims, policy) > worst ? budget_of(dims, policy) : worst;
    if (Mcap < need) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "Mcap = %d but %d rows may be kept", Mcap, need);
    if ((rc = check_ws(ctx, dims, ws, ws_bytes))) return rc;
    cudaStream_t stream = (cudaStream_t)stream_;
    const PrefillWs w = carve(dims, ws);
    if ((rc = upload_small(ctx, w.off, offsets_host, (size_t)dims->B * (dims->S + 1) * 4, stream))) return rc;
    if (token_importance && dims->S > 0) {
        dim3 grid((dims->S + kShotsPerCta - 1) / kShotsPerCta, dims->B * dims->L);
        shot_score_from_tokens_kernel<<<grid, 32 * kShotsPerCta, 0, stream>>>(token_importance, w.off, dims->L, dims->Hkv, dims->N, dims->S, shot_scores);
        LAUNCH_CHECK(ctx);
    }
    if ((rc = run_select(ctx, dims, policy, w, shot_scores, keep, kept_idx, kept_count, Mcap, stream))) return rc;
    if (orc > 0) fail(ctx, orc, "always-kept tokens (%d) exceed the budget (%d) for some prompt", worst, budget_of(dims, policy));
    return orc;
}

// ---- selection without any caller- or library-allocated scratch ------------------------------
// Device copy of the shot boundaries for shotkv_select_shots_static.  It lives in the library
// image: every GPU that loads the library holds these 256 KB until the process exits.
#define SHOTKV_STATIC_OFFSETS_MAX 65536
static __device__ __align__(256) int32_t g_static_offsets[SHOTKV_STATIC_OFFSETS_MAX];

namespace {
// In host code `g_static_offsets` is only a handle; the address kernels can use has to be asked
// for, per device, with that device current.
// The address is kept in the context (a context belongs to one device), so nothing process-wide is
// written: the first call of each context looks it up, with the context's device current.
int static_offsets_ptr(shotkv_ctx* ctx, int32_t** out) {
    if (!ctx->static_offsets) {
        int32_t* p = nullptr;
        CUDA_TRY(ctx, cudaGetSymbolAddress((void**)&p, g_static_offsets));
        if (!p) return fail(ctx, SHOTKV_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
        ctx->static_offsets = p;
    }
    *out = ctx->static_offsets;
    return SHOTKV_OK;
}
}  // namespace

int shotkv_select_shots_static(shotkv_ctx* ctx, const shotkv_dims* dims, const shotkv_policy* policy,
                               const float* token_importance, const int32_t* offsets_host, float* shot_scores,
                               uint8_t* keep, int32_t* kept_idx, int32_t* kept_count, int32_t Mcap, void* stream_) {
    TraceRange trace_("shotkv_select_shots_static");
    int rc = set_device(ctx);
    if (rc) return rc;
    const char* why = "";
    if ((rc = check_dims(dims, &why))) return fail(ctx, rc, "%s", why);
    if ((rc = check_policy_prefill(policy, &why))) return fail(ctx, rc, "%s", why);
    const long long entries = (long long)dims->B * (dims->S + 1);
    if (entries > SHOTKV_STATIC_OFFSETS_MAX)
        return fail(ctx, SHOTKV_ERR_UNSUPPORTED_SHAPE,
                    "B*(S+1) = %lld boundary entries exceed the built-in table of %d; use shotkv_select_shots with a workspace",
                    entries, SHOTKV_STATIC_OFFSETS_MAX);
    int worst = 0;
    const int orc = check_offsets(dims, policy, offsets_host, &worst, &why);
    if (orc < 0) return fail(ctx, orc, "%s", why);
    if (!shot_scores || !keep || !kept_idx || !kept_count) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "output pointers must not be NULL");
    const int need = budget_of(dims, policy) > worst ? budget_of(dims, policy) : worst;
    if (Mcap < need) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "Mcap = %d but %d rows may be kept", Mcap, need);
    cudaStream_t stream = (cudaStream_t)stream_;
    PrefillWs w{};
    if ((rc = static_offsets_ptr(ctx, &w.off))) return rc;
    // every entry the kernels read is overwritten here, so nothing of an earlier call survives
    if ((rc = upload_small(ctx, w.off, offsets_host, (size_t)entries * 4, stream))) return rc;
    if (token_importance && dims->S > 0) {
        dim3 grid((dims->S + kShotsPerCta - 1) / kShotsPerCta, dims->B * dims->L);
        shot_score_from_tokens_kernel<<<grid, 32 * kShotsPerCta, 0, stream>>>(token_importance, w.off, dims->L, dims->Hkv, dims->N, dims->S, shot_scores);
        LAUNCH_CHECK(ctx);
    }
    if ((rc = run_select(ctx, dims, policy, w, shot_scores, keep, kept_idx, kept_count, Mcap, stream))) return rc;
    if (orc > 0) fail(ctx, orc, "always-kept tokens (%d) exceed the budget (%d) for some prompt", worst, budget_of(dims, policy));
    return orc;
}

int shotkv_compact_kv(shotkv_ctx* ctx, const shotkv_dims* dims, const shotkv_bf16* K, const shotkv_bf16* V,
                      const int32_t* kept_idx, const int32_t* kept_count, int32_t Mcap, shotkv_bf16* Kc, shotkv_bf16* Vc,
                      void* stream_) {
    TraceRange trace_("shotkv_compact_kv");
    int rc = set_device(ctx);
    if (rc) return rc;
    const char* why = "";
    if ((rc = check_dims(dims, &why))) return fail(ctx, rc, "%s", why);
    if (!K || !V || !kept_idx || !kept_count || !Kc || !Vc) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "pointers must not be NULL");
    if (Mcap < 1) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "Mcap must be >= 1");
    return run_compact(ctx, dims, K, V, kept_idx, kept_count, Mcap, Kc, Vc, (cudaStream_t)stream_);
}

namespace {
// Called on the caller's stream before a group's scoring pass is enqueued (the host-buffer variant
// copies that group's K there).
using BeforeGroup = std::function<int(const GroupView&, cudaStream_t)>;

int prefill_compress_impl(shotkv_ctx* ctx, const shotkv_dims* dims, const shotkv_policy* policy, const shotkv_bf16* Qwin,
                          const shotkv_bf16* K, const shotkv_bf16* V, const int32_t* offsets_host, float* shot_scores,
                          uint8_t* keep, int32_t* kept_idx, int32_t* kept_count, int32_t Mcap, shotkv_bf16* Kc,
                          shotkv_bf16* Vc, float* token_importance, uint32_t flags, void* ws, size_t ws_bytes,
                          void* stream_, const BeforeGroup* before_group) {
    int rc = set_device(ctx);
    if (rc) return rc;
    const char* why = "";
    if ((rc = check_dims(dims, &why))) return fail(ctx, rc, "%s", why);
    const bool tokens = (flags & SHOTKV_FLAG_TOKEN_IMPORTANCE) != 0;
    if (tokens || token_route(dims)) {
        // per-token importances first (asked for, or many short units): the three public steps in
        // turn; without the flag the importances live in the workspace
        float* imp = token_importance;
        if (!tokens) {
            if ((rc = check_ws(ctx, dims, ws, ws_bytes))) return rc;
            imp = carve(dims, ws).imp;
            prof_begin(ctx);
        }
        if (before_group) {
            const GroupSplit whole{1, dims->B == 1 ? dims->L : dims->B, dims->B == 1};
            if ((rc = (*before_group)(group_view(dims, whole, 0), (cudaStream_t)stream_))) return rc;
        }
        if ((rc = shotkv_prefill_score(ctx, dims, Qwin, K, imp, ws, ws_bytes, stream_)) < 0) return rc;
        if (!tokens) prof_mark(ctx, (cudaStream_t)stream_);
        const int src = shotkv_select_shots(ctx, dims, policy, imp, offsets_host, shot_scores, keep, kept_idx, kept_count,
                                            Mcap, ws, ws_bytes, stream_);
        if (src < 0) return src;
        if (!tokens) prof_mark(ctx, (cudaStream_t)stream_);
        if ((rc = shotkv_compact_kv(ctx, dims, K, V, kept_idx, kept_count, Mcap, Kc, Vc, stream_)) < 0) return rc;
        if (!tokens) prof_mark(ctx, (cudaStream_t)stream_);
        return src;
    }
    if ((rc = check_policy_prefill(policy, &why))) return fail(ctx, rc, "%s", why);
    int worst = 0;
    const int orc = check_offsets(dims, policy, offsets_host, &worst, &why);
    if (orc < 0) return fail(ctx, orc, "%s", why);
    if (!Qwin || !K || !V || !shot_scores || !keep || !kept_idx || !kept_count || !Kc || !Vc)
        return fail(ctx, SHOTKV_ERR_INVALID_ARG, "pointers must not be NULL");
    const int need = budget_of(dims, policy) > worst ? budget_of(dims, policy) : worst;
    if (Mcap < need) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "Mcap = %d but %d rows may be kept", Mcap, need);
    if ((rc = check_ws(ctx, dims, ws, ws_bytes))) return rc;
    cudaStream_t stream = (cudaStream_t)stream_;
    const PrefillWs w = carve(dims, ws);
    const int S = dims->S, R = (dims->H / dims->Hkv) * dims->W, Rpad = rpad_of(dims);
    const size_t S1 = S > 0 ? S : 1, row = dims->d;

    // tables of all prompts once, cut for the work partition of one (full) group
    const GroupSplit gs = plan_groups(ctx, dims, before_group != nullptr);
    const GroupView first = group_view(dims, gs, 0);
    const ChunkPlan plan = plan_chunks(&first.d, ctx->sm_count);
    if ((rc = upload_small(ctx, w.off, offsets_host, (size_t)dims->B * (S + 1) * 4, stream))) return rc;
    int P = 0;
    if ((rc = prepare_pieces(ctx, dims, offsets_host, plan, w, &P, stream))) return rc;
    const size_t msm = ((size_t)P + 2 * Rpad) * 4;     // shot_mass_kernel: row statistics and one mass per piece
    if (S > 0) {
        if (msm > kBigSmem) return fail(ctx, SHOTKV_ERR_UNSUPPORTED_SHAPE, "too many shots for the single-pass path (S = %d)", S);
    }
    prof_begin(ctx);
    const bool forked = gs.n > 1;
    cudaStream_t tail = forked ? ctx->aux : stream;
    // Once a group has been handed to the second stream, an early return must still order that
    // work before whatever the caller enqueues next on `stream`.
    bool handed = false;
    auto bail = [&](int code) {
        if (forked && handed && cudaEventRecord(ctx->ev_join, tail) == cudaSuccess) cudaStreamWaitEvent(stream, ctx->ev_join, 0);
        return code;
    };
    for (int g = 0; g < gs.n; ++g) {
        const GroupView v = group_view(dims, gs, g);
        const PrefillWs wg = group_ws(w, dims, v, g, P);
        const shotkv_dims* dg = &v.d;
        const int Ug = dg->B * dg->L * dg->Hkv;
        const shotkv_bf16* Kg = K + v.u0 * dims->N * row;
        const shotkv_bf16* Vg = V + v.u0 * dims->N * row;
        float* scores_g = shot_scores + v.bl0 * S1;
        int32_t* idx_g = kept_idx + v.bl0 * (size_t)Mcap;
        int32_t* count_g = kept_count + v.bl0;
        if (before_group && (rc = (*before_group)(v, stream))) return bail(rc);
        prof_gmark(ctx, g, 0, stream);
        if ((rc = launch_score_tc(ctx, dg, Qwin + v.bl0 * dims->H * dims->W * row, Kg, wg, P, plan, stream))) return bail(rc);
        prof_gmark(ctx, g, 1, stream);
        if (forked) {
            if (cudaEventRecord(ctx->ev_fork[g], stream) != cudaSuccess || cudaStreamWaitEvent(tail, ctx->ev_fork[g], 0) != cudaSuccess)
                return bail(fail(ctx, SHOTKV_ERR_CUDA, "could not hand a group of units to the second stream"));
            handed = true;
        }
        prof_gmark(ctx, g, 2, tail);
        if (S > 0) {
            const PartialView pv = partial_view(ctx, dg, wg, P, plan);
            if (Rpad == 128)
                shot_mass_kernel<128><<<Ug, 128, msm, tail>>>(pv, wg.piece_seg, R, dg->L, dg->Hkv, S, wg.unit_shot);
            else
                shot_mass_kernel<256><<<Ug, 256, msm, tail>>>(pv, wg.piece_seg, R, dg->L, dg->Hkv, S, wg.unit_shot);
            ctx->launches += 1;
            if (cudaGetLastError() != cudaSuccess) return bail(fail(ctx, SHOTKV_ERR_CUDA, "per-shot reduction failed to launch"));
            shot_score_from_mass_kernel<<<dg->B * dg->L, 128, 0, tail>>>(wg.unit_shot, wg.off, dg->L, dg->Hkv, S, scores_g);
            ctx->launches += 1;
            if (cudaGetLastError() != cudaSuccess) return bail(fail(ctx, SHOTKV_ERR_CUDA, "per-shot score kernel failed to launch"));
        }
        prof_gmark(ctx, g, 3, tail);
        if ((rc = run_select(ctx, dg, policy, wg, scores_g, keep + v.bl0 * S1, idx_g, count_g, Mcap, tail))) return bail(rc);
        prof_gmark(ctx, g, 4, tail);
        if ((rc = run_compact(ctx, dg, Kg, Vg, idx_g, count_g, Mcap, Kc + v.u0 * (size_t)Mcap * row, Vc + v.u0 * (size_t)Mcap * row, tail))) return bail(rc);
        prof_gmark(ctx, g, 5, tail);
    }
    if (forked) {
        CUDA_TRY(ctx, cudaEventRecord(ctx->ev_join, tail));
        CUDA_TRY(ctx, cudaStreamWaitEvent(stream, ctx->ev_join, 0));
    }
    if (orc > 0) fail(ctx, orc, "always-kept tokens (%d) exceed the budget (%d) for some prompt", worst, budget_of(dims, policy));
    return orc;
}
}  // namespace

int shotkv_prefill_compress(shotkv_ctx* ctx, const shotkv_dims* dims, const shotkv_policy* policy, const shotkv_bf16* Qwin,
                            const shotkv_bf16* K, const shotkv_bf16* V, const int32_t* offsets_host, float* shot_scores,
                            uint8_t* keep, int32_t* kept_idx, int32_t* kept_count, int32_t Mcap, shotkv_bf16* Kc,
                            shotkv_bf16* Vc, float* token_importance, uint32_t flags, void* ws, size_t ws_bytes,
                            void* stream_) {
    TraceRange trace_("shotkv_prefill_compress");
    return prefill_compress_impl(ctx, dims, policy, Qwin, K, V, offsets_host, shot_scores, keep, kept_idx, kept_count, Mcap, Kc,
                                 Vc, token_importance, flags, ws, ws_bytes, stream_, nullptr);
}

// ---- host-buffer variant -------------------------------------------------------------------
namespace {
struct HostArena {
    shotkv_bf16 *Q, *K, *V, *Kc, *Vc;
    float* scores;
    uint8_t* keep;
    int32_t *idx, *count;
    void* ws;
    size_t ws_bytes, total;
};
HostArena carve_host(const shotkv_dims* d, int32_t Mcap, void* base) {
    HostArena a{};
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o += align_up(bytes); return (unsigned char*)base + at; };
    const size_t BL = (size_t)d->B * d->L, U = BL * d->Hkv;
    a.Q = (shotkv_bf16*)take(BL * d->H * d->W * d->d * 2);
    a.K = (shotkv_bf16*)take(U * d->N * d->d * 2);
    a.V = (shotkv_bf16*)take(U * d->N * d->d * 2);
    a.Kc = (shotkv_bf16*)take(U * (size_t)Mcap * d->d * 2);
    a.Vc = (shotkv_bf16*)take(U * (size_t)Mcap * d->d * 2);
    a.scores = (float*)take(BL * (size_t)(d->S > 0 ? d->S : 1) * 4);
    a.keep = (uint8_t*)take(BL * (size_t)(d->S > 0 ? d->S : 1));
    a.idx = (int32_t*)take(BL * (size_t)Mcap * 4);
    a.count = (int32_t*)take(BL * 4);
    a.ws_bytes = shotkv_workspace_bytes(d);
    a.ws = take(a.ws_bytes);
    a.total = o;
    return a;
}
}  // namespace

size_t shotkv_host_arena_bytes(const shotkv_dims* dims, int32_t Mcap) {
    const char* why = "";
    if (check_dims(dims, &why) || Mcap < 1) return 0;
    return carve_host(dims, Mcap, nullptr).total;
}

int shotkv_prefill_compress_host(shotkv_ctx* ctx, const shotkv_dims* dims, const shotkv_policy* policy,
                                 const shotkv_bf16* Qwin_host, const shotkv_bf16* K_host, const shotkv_bf16* V_host,
                                 const int32_t* offsets_host, float* shot_scores_host, uint8_t* keep_host,
                                 int32_t* kept_idx_host, int32_t* kept_count_host, int32_t Mcap, shotkv_bf16* Kc_host,
                                 shotkv_bf16* Vc_host, void* arena, size_t arena_bytes, void* stream_) {
    TraceRange trace_("shotkv_prefill_compress_host");
    int rc = set_device(ctx);
    if (rc) return rc;
    const char* why = "";
    if ((rc = check_dims(dims, &why))) return fail(ctx, rc, "%s", why);
    if (!Qwin_host || !K_host || !V_host) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "host inputs must not be NULL");
    if (Mcap < 1) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "Mcap must be >= 1");
    if (!arena || (uintptr_t)arena % 256) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "arena must be a 256-byte aligned device buffer");
    const HostArena a = carve_host(dims, Mcap, arena);
    if (arena_bytes < a.total) return fail(ctx, SHOTKV_ERR_WORKSPACE_TOO_SMALL, "arena has %zu bytes, %zu needed", arena_bytes, a.total);
    cudaStream_t stream = (cudaStream_t)stream_;
    const size_t BL = (size_t)dims->B * dims->L, U = BL * dims->Hkv;
    // Page-locked host buffers are addressable from the device.  V is only ever gathered (the rows
    // of the kept tokens), so a page-locked V is read in place by the compaction kernel instead of
    // being copied whole, and page-locked Kc/Vc are written in place by it.  Pageable buffers take
    // the staged copies through the arena.
    auto device_alias = [](const void* host) -> void* {
        if (!host) return nullptr;
        cudaPointerAttributes at{};
        if (cudaPointerGetAttributes(&at, host) != cudaSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
    };
    const shotkv_bf16* V_in = (const shotkv_bf16*)device_alias(V_host);
    shotkv_bf16* Kc_out = (shotkv_bf16*)device_alias(Kc_host);
    shotkv_bf16* Vc_out = (shotkv_bf16*)device_alias(Vc_host);
    if (((uintptr_t)V_in | (uintptr_t)Kc_out | (uintptr_t)Vc_out) & 15) V_in = nullptr, Kc_out = Vc_out = nullptr;
    CUDA_TRY(ctx, cudaMemcpyAsync(a.Q, Qwin_host, BL * dims->H * dims->W * dims->d * 2, cudaMemcpyHostToDevice, stream));
    // K goes up one group of units at a time, just ahead of that group's scoring pass, so that the
    // copies of later groups run beside the gathers and write-backs of earlier ones
    const size_t unit_elems = (size_t)dims->N * dims->d;
    const BeforeGroup copy_k = [&](const GroupView& v, cudaStream_t s) -> int {
        const size_t units = (size_t)v.d.B * v.d.L * v.d.Hkv;
        CUDA_TRY(ctx, cudaMemcpyAsync(a.K + v.u0 * unit_elems, K_host + v.u0 * unit_elems, units * unit_elems * 2, cudaMemcpyHostToDevice, s));
        return SHOTKV_OK;
    };
    if (!V_in) {
        CUDA_TRY(ctx, cudaMemcpyAsync(a.V, V_host, U * dims->N * dims->d * 2, cudaMemcpyHostToDevice, stream));
        V_in = a.V;
    }
    const int prc = prefill_compress_impl(ctx, dims, policy, a.Q, a.K, V_in, offsets_host, a.scores, a.keep, a.idx, a.count,
                                          Mcap, Kc_out ? Kc_out : a.Kc, Vc_out ? Vc_out : a.Vc, nullptr, 0, a.ws,
                                          a.ws_bytes, stream_, &copy_k);
    if (prc < 0) return prc;
    const size_t S1 = dims->S > 0 ? dims->S : 1;
    if (shot_scores_host) CUDA_TRY(ctx, cudaMemcpyAsync(shot_scores_host, a.scores, BL * S1 * 4, cudaMemcpyDeviceToHost, stream));
    if (keep_host) CUDA_TRY(ctx, cudaMemcpyAsync(keep_host, a.keep, BL * S1, cudaMemcpyDeviceToHost, stream));
    if (kept_idx_host) CUDA_TRY(ctx, cudaMemcpyAsync(kept_idx_host, a.idx, BL * (size_t)Mcap * 4, cudaMemcpyDeviceToHost, stream));
    if (kept_count_host) CUDA_TRY(ctx, cudaMemcpyAsync(kept_count_host, a.count, BL * 4, cudaMemcpyDeviceToHost, stream));
    if (Kc_host && !Kc_out) CUDA_TRY(ctx, cudaMemcpyAsync(Kc_host, a.Kc, U * (size_t)Mcap * dims->d * 2, cudaMemcpyDeviceToHost, stream));
    if (Vc_host && !Vc_out) CUDA_TRY(ctx, cudaMemcpyAsync(Vc_host, a.Vc, U * (size_t)Mcap * dims->d * 2, cudaMemcpyDeviceToHost, stream));
    return prc;
}

// ---- decode ---------------------------------------------------------------------------------
size_t shotkv_decode_workspace_bytes(const shotkv_dims* dims, int32_t Dcap) {
    if (!dims || Dcap < 1 || dims->B < 1 || dims->L < 1 || dims->Hkv < 1) return 0;
    const size_t BL = (size_t)dims->B * dims->L;
    return align_up(BL * dims->Hkv * (size_t)Dcap * 4) + align_up(BL * (size_t)Dcap * 4);
}

int32_t shotkv_decode_capacity(const shotkv_policy* policy, int32_t steps) {
    if (!policy || steps < 0 || policy->recompress_every < 1 || !(policy->r_d >= 0.f) || policy->protect_recent < 0)
        return SHOTKV_ERR_INVALID_ARG;
    // replay the host-side counters
    int n = 0, worst = 1;
    for (int T = 1; T <= steps; ++T) {
        ++n;
        if (n > worst) worst = n;
        if (T % policy->recompress_every == 0) {
            int k = (int)std::floor((double)policy->r_d * (double)T);
            const int prot = policy->protect_recent < T ? policy->protect_recent : T;
            if (k < prot) k = prot;
            if (k < n) n = k;
        }
    }
    return worst;
}

int shotkv_decode_init(shotkv_ctx* ctx, const shotkv_dims* dims, const shotkv_policy* policy, int32_t Dcap, int32_t Mcap,
                       shotkv_bf16* Kd, shotkv_bf16* Vd, float* acc, int32_t* born, void* ws, size_t ws_bytes,
                       shotkv_decode_state* state) {
    if (!ctx) return SHOTKV_ERR_INVALID_ARG;
    if (!dims || !policy || !state) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "dims, policy and state must not be NULL");
    if (dims->B < 1 || dims->L < 1 || dims->H < 1 || dims->Hkv < 1 || dims->H % dims->Hkv)
        return fail(ctx, SHOTKV_ERR_INVALID_ARG, "B, L, H, Hkv must be >= 1 and H a multiple of Hkv");
    if (dims->d != 64 && dims->d != 128) return fail(ctx, SHOTKV_ERR_UNSUPPORTED_SHAPE, "head dimension must be 64 or 128");
    if (dims->H / dims->Hkv > 8) return fail(ctx, SHOTKV_ERR_UNSUPPORTED_SHAPE, "decode supports H/Hkv <= 8");
    if (!(policy->r_d >= 0.f) || !std::isfinite(policy->r_d)) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "r_d must be finite and >= 0");
    if (policy->recompress_every < 1) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "recompress_every must be >= 1");
    if (policy->protect_recent < 0) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "protect_recent must be >= 0");
    if (Dcap < 1 || Dcap > 4096) return fail(ctx, SHOTKV_ERR_UNSUPPORTED_SHAPE, "Dcap must be in [1, 4096]");
    if (Mcap < 0) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "Mcap must be >= 0");
    if (!Kd || !Vd || !acc || !born || !ws) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "device pointers must not be NULL");
    if (ws_bytes < shotkv_decode_workspace_bytes(dims, Dcap))
        return fail(ctx, SHOTKV_ERR_WORKSPACE_TOO_SMALL, "decode workspace has %zu bytes, %zu needed", ws_bytes,
                    shotkv_decode_workspace_bytes(dims, Dcap));
    memset(state, 0, sizeof(*state));
    state->dims = *dims;
    state->policy = *policy;
    state->Dcap = Dcap;
    state->Mcap = Mcap;
    state->Kd = Kd; state->Vd = Vd; state->acc = acc; state->born = born;
    state->ws = ws; state->ws_bytes = ws_bytes;
    return SHOTKV_OK;
}

}  // extern "C"

namespace {

template <int D>
int launch_decode_attend(shotkv_ctx* ctx, const DecodeParams& p, int U, cudaStream_t stream) {
    using Cfg = AttendCfg<D>;
    const size_t smem = ((size_t)8 * p.Dcap + Cfg::kWarps * 8 * 2 + 16) * 4 + Cfg::kRingBytes;
    if (smem > kBigSmem) return fail(ctx, SHOTKV_ERR_UNSUPPORTED_SHAPE, "Dcap too large for the attention-output step");
    decode_attend_kernel<D><<<U, Cfg::kWarps * 32, smem, stream>>>(p);
    return SHOTKV_OK;
}

// One decode step; with `attn_out` the score kernel is the variant that also writes the attention output.
int decode_step_impl(shotkv_ctx* ctx, shotkv_decode_state* st, const shotkv_bf16* q, const shotkv_bf16* k_new,
                     const shotkv_bf16* v_new, const shotkv_bf16* Kc, const shotkv_bf16* Vc, const int32_t* kept_count,
                     float* attn_out, void* stream_) {
    int rc = set_device(ctx);
    if (rc) return rc;
    if (!st || !q || !k_new || !v_new || !kept_count) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "pointers must not be NULL");
    if (st->Mcap > 0 && !Kc) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "Kc must not be NULL when Mcap > 0");
    if (attn_out && st->Mcap > 0 && !Vc) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "Vc must not be NULL when Mcap > 0");
    if (st->n_dec + 1 > st->Dcap) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "decode region full: n_dec = %d, Dcap = %d", st->n_dec, st->Dcap);
    cudaStream_t stream = (cudaStream_t)stream_;
    const shotkv_dims& d = st->dims;
    const int BL = d.B * d.L, U = BL * d.Hkv;
    float* partial = (float*)st->ws;
    int* keep_pos = (int*)((unsigned char*)st->ws + align_up((size_t)U * st->Dcap * 4));

    DecodeParams p{};
    p.q = (const __nv_bfloat16*)q; p.k_new = (const __nv_bfloat16*)k_new; p.v_new = (const __nv_bfloat16*)v_new;
    p.Kc = (const __nv_bfloat16*)Kc; p.kept_count = kept_count;
    p.Kd = (__nv_bfloat16*)st->Kd; p.Vd = (__nv_bfloat16*)st->Vd; p.partial = partial;
    p.H = d.H; p.Hkv = d.Hkv; p.G = d.H / d.Hkv; p.Mcap = st->Mcap; p.Dcap = st->Dcap; p.n_old = st->n_dec;
    p.scale_log2 = kLog2e / sqrtf((float)d.d);
    p.Vc = (const __nv_bfloat16*)Vc; p.out = attn_out;
    const size_t smem = (size_t)8 * st->Dcap * 4 + (8 * 8 * 2 + 16) * 4;
    prof_begin(ctx);
    prof_mark(ctx, stream);
    if (attn_out) {
        rc = d.d == 128 ? launch_decode_attend<128>(ctx, p, U, stream) : launch_decode_attend<64>(ctx, p, U, stream);
        if (rc) return rc;
    } else if (d.d == 128) {
        decode_score_kernel<128><<<U, 256, smem, stream>>>(p);
    } else {
        decode_score_kernel<64><<<U, 256, smem, stream>>>(p);
    }
    LAUNCH_CHECK(ctx);
    prof_mark(ctx, stream);
    decode_accumulate_kernel<<<BL, 128, 0, stream>>>(partial, d.Hkv, st->Dcap, st->n_dec, st->T, st->acc, st->born);
    LAUNCH_CHECK(ctx);
    st->n_dec += 1;
    st->T += 1;
    if (st->T % st->policy.recompress_every == 0) {
        const int n = st->n_dec;
        int k = (int)std::floor((double)st->policy.r_d * (double)st->T);
        // entries of the last protect_recent steps are all still present (they were protected at every
        // earlier eviction too) and are kept whatever their score; the others share what is left of k
        const int prot = st->policy.protect_recent < st->T ? st->policy.protect_recent : st->T;
        if (k < prot) k = prot;
        if (k > n) k = n;
        if (k < n) {
            const size_t rs = (size_t)n * 16 + (kSelectThreads + 1) * 4 + 16;
            decode_rank_kernel<<<BL, kSelectThreads, rs, stream>>>(st->acc, st->born, st->Dcap, n, k,
                                                                   prot > 0 ? st->T - prot : 0x7fffffff, keep_pos);
            LAUNCH_CHECK(ctx);
            if (k > 0) {
                dim3 grid(U, 2);
                if (d.d == 128)
                    decode_compact_kernel<128><<<grid, 256, 0, stream>>>((__nv_bfloat16*)st->Kd, (__nv_bfloat16*)st->Vd, keep_pos, d.Hkv, st->Dcap, k);
                else
                    decode_compact_kernel<64><<<grid, 256, 0, stream>>>((__nv_bfloat16*)st->Kd, (__nv_bfloat16*)st->Vd, keep_pos, d.Hkv, st->Dcap, k);
                LAUNCH_CHECK(ctx);
            }
            st->n_dec = k;
        }
    }
    prof_mark(ctx, stream);
    return SHOTKV_OK;
}

}  // namespace

extern "C" {

int shotkv_decode_step(shotkv_ctx* ctx, shotkv_decode_state* st, const shotkv_bf16* q, const shotkv_bf16* k_new,
                       const shotkv_bf16* v_new, const shotkv_bf16* Kc, const int32_t* kept_count, void* stream) {
    TraceRange trace_("shotkv_decode_step");
    return decode_step_impl(ctx, st, q, k_new, v_new, Kc, nullptr, kept_count, nullptr, stream);
}

int shotkv_decode_step_attend(shotkv_ctx* ctx, shotkv_decode_state* st, const shotkv_bf16* q, const shotkv_bf16* k_new,
                              const shotkv_bf16* v_new, const shotkv_bf16* Kc, const shotkv_bf16* Vc,
                              const int32_t* kept_count, float* attn_out, void* stream) {
    TraceRange trace_("shotkv_decode_step_attend");
    if (!attn_out) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "attn_out must not be NULL");
    return decode_step_impl(ctx, st, q, k_new, v_new, Kc, Vc, kept_count, attn_out, stream);
}

int32_t shotkv_plan_pieces(const shotkv_dims* dims, const int32_t* offsets_host, int32_t sm_count, int32_t* nchunk,
                           int32_t* chunk_keys, int32_t* pieces_out, int32_t cap) {
    const char* why = "";
    int rc = check_dims(dims, &why);
    if (rc) return rc;
    if (offsets_host && (rc = check_offsets(dims, nullptr, offsets_host, nullptr, &why)) < 0) return rc;
    if (sm_count < 1) return SHOTKV_ERR_INVALID_ARG;
    const ChunkPlan plan = plan_chunks(dims, sm_count);
    std::vector<int2> pieces;
    std::vector<int> seg, chunk_first;
    const int P = build_pieces(dims, offsets_host, plan, pieces, seg, chunk_first);
    if (nchunk) *nchunk = plan.nchunk;
    if (chunk_keys) *chunk_keys = plan.chunk_keys;
    if (pieces_out) {
        if (cap < P) return SHOTKV_ERR_INVALID_ARG;
        for (int b = 0; b < dims->B; ++b)
            for (int i = 0; i < P; ++i) {
                int32_t* o = pieces_out + ((size_t)b * cap + i) * 3;
                o[0] = pieces[(size_t)b * P + i].x;
                o[1] = pieces[(size_t)b * P + i].y;
                o[2] = seg[(size_t)b * P + i];
            }
    }
    return P;
}

// ---- instrumentation ------------------------------------------------------------------------
int shotkv_set_scoring_mode(shotkv_ctx* ctx, int mode) {
    if (!ctx) return SHOTKV_ERR_INVALID_ARG;
    if (mode != SHOTKV_SCORING_FAST && mode != SHOTKV_SCORING_EXACT)
        return fail(ctx, SHOTKV_ERR_INVALID_ARG, "scoring mode must be SHOTKV_SCORING_FAST or SHOTKV_SCORING_EXACT");
    ctx->scoring_mode = mode;
    return SHOTKV_OK;
}

int shotkv_set_wait_limit(shotkv_ctx* ctx, int64_t cycles) {
    if (!ctx) return SHOTKV_ERR_INVALID_ARG;
    if (cycles < 0) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "wait limit must be >= 0 cycles (0 restores the default)");
    ctx->wait_cycles = cycles == 0 ? tc::kWaitCycles : (long long)cycles;
    return SHOTKV_OK;
}

int shotkv_selftest_bounded_wait(shotkv_ctx* ctx, int64_t limit_cycles, int32_t* report, void* stream_) {
    TraceRange trace_("shotkv_selftest_bounded_wait");
    int rc = set_device(ctx);
    if (rc) return rc;
    if (!report) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "report must not be NULL");
    if (limit_cycles < 1000 || limit_cycles > 1000000000LL)
        return fail(ctx, SHOTKV_ERR_INVALID_ARG, "self-test limit must be between 1e3 and 1e9 cycles");
    cudaStream_t stream = (cudaStream_t)stream_;
    for (int i = 0; i < 4; ++i) ((volatile int*)ctx->err_host)[2 + i] = -1;
    bounded_wait_selftest_kernel<<<1, 64, 0, stream>>>((long long)limit_cycles, ctx->err_dev, ctx->err_dev + 2);
    LAUNCH_CHECK(ctx);
    CUDA_TRY(ctx, cudaStreamSynchronize(stream));
    for (int i = 0; i < 4; ++i) report[i] = ((volatile int*)ctx->err_host)[2 + i];
    return SHOTKV_OK;
}

int shotkv_set_pipeline_groups(shotkv_ctx* ctx, int groups) {
    if (!ctx) return SHOTKV_ERR_INVALID_ARG;
    if (groups < 0 || groups > kMaxGroups)
        return fail(ctx, SHOTKV_ERR_INVALID_ARG, "pipeline groups must be 0 (automatic) or 1..%d", kMaxGroups);
    ctx->pipeline_groups = groups;
    return SHOTKV_OK;
}

int shotkv_profile_enable(shotkv_ctx* ctx, int enable) {
    int rc = set_device(ctx);
    if (rc) return rc;
    if (enable && !ctx->prof_ev[0][0]) {
        for (int i = 0; i < kProfSlots; ++i) {
            for (int j = 0; j < 5; ++j) CUDA_TRY(ctx, cudaEventCreate(&ctx->prof_ev[i][j]));
            for (int g = 0; g < kMaxGroups; ++g)
                for (int j = 0; j < 6; ++j) CUDA_TRY(ctx, cudaEventCreate(&ctx->prof_gev[i][g][j]));
        }
    }
    ctx->prof = enable != 0;
    ctx->prof_calls = 0;
    return SHOTKV_OK;
}

int shotkv_profile_read(shotkv_ctx* ctx, int calls_back, float* stage_ms) {
    int rc = set_device(ctx);
    if (rc) return rc;
    if (!stage_ms || calls_back < 0 || calls_back >= kProfSlots || calls_back >= ctx->prof_calls)
        return fail(ctx, SHOTKV_ERR_INVALID_ARG, "no profiled call %d calls back", calls_back);
    const int slot = (ctx->prof_calls - 1 - calls_back) % kProfSlots;
    const int m = ctx->prof_marks[slot];
    for (int i = 0; i < 4; ++i) stage_ms[i] = -1.f;
    if (const int ng = ctx->prof_groups[slot]) {
        // pipelined fused call: each stage's time summed over the groups (the stages of different
        // groups overlap, so the sum may exceed the call's wall time)
        CUDA_TRY(ctx, cudaEventSynchronize(ctx->prof_gev[slot][ng - 1][5]));
        static const int from[4] = {0, 2, 3, 4};
        for (int i = 0; i < 4; ++i) {
            float sum = 0.f;
            for (int g = 0; g < ng; ++g) {
                float ms = 0.f;
                CUDA_TRY(ctx, cudaEventElapsedTime(&ms, ctx->prof_gev[slot][g][from[i]], ctx->prof_gev[slot][g][from[i] + 1]));
                sum += ms;
            }
            stage_ms[i] = sum;
        }
        return 4;
    }
    if (m < 2) return fail(ctx, SHOTKV_ERR_INVALID_ARG, "that call recorded no stages");
    CUDA_TRY(ctx, cudaEventSynchronize(ctx->prof_ev[slot][m - 1]));
    for (int i = 0; i + 1 < m; ++i) CUDA_TRY(ctx, cudaEventElapsedTime(&stage_ms[i], ctx->prof_ev[slot][i], ctx->prof_ev[slot][i + 1]));
    return m - 1;
}

uint64_t shotkv_launch_count(const shotkv_ctx* ctx) { return ctx ? ctx->launches : 0; }

int shotkv_last_scoring_clock(const shotkv_ctx* ctx, int64_t* cycles, int64_t* nanoseconds) {
    if (!ctx || !ctx->err_host || !cycles || !nanoseconds) return SHOTKV_ERR_INVALID_ARG;
    const volatile long long* w = (const volatile long long*)(ctx->err_host + 8);
    *cycles = (int64_t)(w[2] - w[0]);
    *nanoseconds = (int64_t)(w[3] - w[1]);
    return SHOTKV_OK;
}

uint64_t shotkv_repaired_items(const shotkv_ctx* ctx) {
    return ctx && ctx->err_host ? (uint64_t)(unsigned)((volatile int*)ctx->err_host)[1] : 0;
}

}  // extern "C"
