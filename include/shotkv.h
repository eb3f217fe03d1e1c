/*
 * shotkv.h -- C ABI of the ShotKV hot path for NVIDIA B200 (sm_100a).
 *
 * ShotKV (arXiv 2502.01941, Section 5.1 and Algorithm 1) compresses the KV cache
 * of a few-shot prompt once after prefill, keeping whole shots ("semantic units")
 * ranked by the attention they receive, and compresses the decode-side cache
 * token by token while generating.  This library is that path and nothing else.
 *
 * Conventions for every call
 *   - "device" pointers are CUDA global memory of the context's device, "host"
 *     pointers are ordinary process memory.  The caller owns every buffer,
 *     workspaces included; the library owns only the shotkv_ctx.
 *   - bf16 tensors are raw 16-bit patterns (shotkv_bf16).  Rows of d contiguous
 *     elements; all tensors dense in the index order written beside them; base
 *     addresses 16-byte aligned.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = the
 *     legacy default stream); calls return without synchronising unless stated.
 *   - Return value: 0 = ok, negative = error (nothing useful was enqueued),
 *     positive = warning (the work was enqueued).  shotkv_last_error() gives text.
 *   - There is no CPU fallback: without a CUDA device every compute call fails.
 *
 * Index names: B prompts, L layers, H query heads, Hkv KV heads (G = H/Hkv),
 * d head dimension (64 or 128), N prompt tokens, W observation-window rows
 * (the last W prompt positions), S shots.  Shot i covers tokens
 * [off[i], off[i+1]) and has k_i = off[i+1]-off[i] >= 1 tokens; tokens before
 * off[0] and from off[S] on (the question, which contains the window) are
 * always kept and count against the budget.
 */
#ifndef SHOTKV_H_
#define SHOTKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define SHOTKV_API __attribute__((visibility("default")))
#else
#define SHOTKV_API
#endif

typedef struct shotkv_ctx shotkv_ctx;
typedef uint16_t shotkv_bf16;

typedef struct {
    int32_t B, L, H, Hkv, d, N, W, S;
} shotkv_dims;
/* The paper selects per layer: one kept set for all KV heads of a layer (Section 5.1).  A kept set
 * per KV head -- every head ranks the shots by the attention its own query group pays them, and
 * the compressed caches become ragged across heads -- needs no other call: with the dense layouts
 * above, a tensor of L layers x Hkv heads is also a tensor of L*Hkv "layers" of one head, so pass
 *   { B, L * Hkv, H / Hkv, 1, d, N, W, S }
 * with the same pointers.  Every per-layer output then has one entry per (layer, KV head).  */

typedef struct {
    float   r_p;              /* prefill ratio: N_budget = floor(r_p * N) tokens per layer        */
    int32_t select_mode;      /* 0: stop at the first shot that overflows; 1: skip it and go on   */
    float   r_d;              /* decode ratio: k = floor(r_d * T) after T generated tokens        */
    int32_t recompress_every; /* decode: evict every this many steps (1 = every step)             */
    int32_t protect_recent;   /* decode: entries of the last this many steps are never evicted;   */
                              /* 0 = the paper's rule, which protects nothing                     */
} shotkv_policy;

enum {
    SHOTKV_OK = 0,
    SHOTKV_ERR_INVALID_ARG = -1,
    SHOTKV_ERR_UNSUPPORTED_SHAPE = -2,
    SHOTKV_ERR_BAD_OFFSETS = -3,          /* not increasing, empty shot, off[0] < 0 or off[S] > N-W  */
    SHOTKV_ERR_WORKSPACE_TOO_SMALL = -4,
    SHOTKV_ERR_CUDA = -5,
    SHOTKV_ERR_TIMEOUT = -6,              /* a bounded device-side wait gave up                     */
    SHOTKV_WARN_BUDGET_BELOW_ALWAYS_KEPT = 1 /* some prompt's always-kept tokens exceed floor(r_p*N);
                                                only they are kept for that prompt                  */
};

/* Bit set in `flags` of shotkv_prefill_compress. */
#define SHOTKV_FLAG_TOKEN_IMPORTANCE 1u   /* also produce per-token importance (two passes over K) */

/* ---- context ------------------------------------------------------------------------------- */

/* Creates a context bound to CUDA device `device`.  Fails with SHOTKV_ERR_CUDA when there is no
 * such device or it is not compute capability 10.x.  */
SHOTKV_API int shotkv_create(shotkv_ctx** ctx, int device);
SHOTKV_API void shotkv_destroy(shotkv_ctx* ctx);
/* Text of the last error or warning recorded on this context (never NULL; "" if none). */
SHOTKV_API const char* shotkv_last_error(const shotkv_ctx* ctx);
/* Library version string. */
SHOTKV_API const char* shotkv_version(void);

/* ---- host helpers (no GPU needed) ---------------------------------------------------------- */

/* N_budget = floor(r_p * N), the product taken in double with r_p as the float it is
 * (Section 5.1: budget r_p x |KV_prefill|, |KV_prefill| = all N prompt tokens).  */
SHOTKV_API int32_t shotkv_budget_tokens(const shotkv_dims* dims, const shotkv_policy* policy);
/* Rows to allocate per (b,l[,hkv]) for kept_idx / Kc / Vc: max(N_budget, largest always-kept
 * count over the B prompts).  offsets_host [B][S+1].  Negative error code on bad input.  */
SHOTKV_API int32_t shotkv_kept_capacity(const shotkv_dims* dims, const shotkv_policy* policy,
                             const int32_t* offsets_host);
/* Checks shapes and offsets exactly as the compute calls do.  Returns 0, a negative error, or
 * SHOTKV_WARN_BUDGET_BELOW_ALWAYS_KEPT.  policy and offsets_host may be NULL to check dims only. */
SHOTKV_API int shotkv_validate(const shotkv_dims* dims, const shotkv_policy* policy,
                    const int32_t* offsets_host);
/* Bytes of device workspace that the prefill calls below need for `dims` (any of them; one
 * buffer of this size serves all).  0 on invalid dims.  */
SHOTKV_API size_t shotkv_workspace_bytes(const shotkv_dims* dims);

/* ---- prefill (Algorithm 1, Phase 1) -------------------------------------------------------- */

/* Window attention and column-sum: the alpha of the prefill score equation (Section 5.1).
 * For every (b, l, kv head g) the R = G*W window rows (heads g*G..g*G+G-1, positions N-W..N-1)
 * attend causally to the prompt keys with scale 1/sqrt(d); every row is a softmax over the keys at
 * or before its own position; token_importance[b][l][g][t] is the sum of column t over those rows.
 *   Qwin  device [B][L][H][W][d] bf16      K  device [B][L][Hkv][N][d] bf16
 *   token_importance  device [B][L][Hkv][N] f32 (written in full)
 *   ws    device workspace of >= shotkv_workspace_bytes(dims) bytes, 256-byte aligned
 * Supported: d in {64,128}, G*W <= 256, W <= N.  */
SHOTKV_API int shotkv_prefill_score(shotkv_ctx* ctx, const shotkv_dims* dims,
                         const shotkv_bf16* Qwin, const shotkv_bf16* K,
                         float* token_importance, void* ws, size_t ws_bytes, void* stream);

/* Per-shot score and whole-shot selection (prefill score equation, TopK equation and its budget
 * constraint in Section 5.1; "sort ... select shots until" in Algorithm 1).
 *   Score(s_i) = (1/k_i) * sum_{t in s_i} sum_{g} token_importance[b][l][g][t]      per (b, l)
 * Shots are ordered by (score descending, index ascending) and kept per `select_mode` while the
 * kept shot tokens fit floor(r_p*N) minus the always-kept tokens.  Scores must be finite.
 *   token_importance device [B][L][Hkv][N] f32, or NULL to rank the shot_scores already in place
 *   offsets_host     host   [B][S+1] int32 (validated; uploaded into ws on `stream`)
 *   shot_scores      device [B][L][S] f32   (output; input when token_importance is NULL)
 *   keep             device [B][L][S] u8    1 = shot kept
 *   kept_idx         device [B][L][Mcap] i32 kept token positions ascending, -1 beyond kept_count
 *   kept_count       device [B][L] i32
 *   Mcap >= shotkv_kept_capacity(...).  */
SHOTKV_API int shotkv_select_shots(shotkv_ctx* ctx, const shotkv_dims* dims, const shotkv_policy* policy,
                        const float* token_importance, const int32_t* offsets_host,
                        float* shot_scores, uint8_t* keep, int32_t* kept_idx, int32_t* kept_count,
                        int32_t Mcap, void* ws, size_t ws_bytes, void* stream);

/* shotkv_select_shots for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a packaging variant, the arithmetic is that of shotkv_select_shots).
 * Some hosts of this library may not call cudaMalloc at the point where they compress a prompt:
 * an inference server that handed all of HBM to its own pool at start-up, a plug-in running
 * inside another runtime's stream callback or memory-frozen region, a real-time loop that bans
 * allocator calls.  shotkv_select_shots needs a caller-supplied workspace only to hold the device
 * copy of the shot boundaries; here that copy lives in a fixed table inside the library image
 * (SHOTKV_STATIC_OFFSETS_MAX = 65536 int32 entries, 256 KB, resident on every GPU that loads the
 * library until the process exits).  The call performs no cudaMalloc/cudaFree and uses no
 * allocating library routine.
 *   - Limit: B*(S+1) <= 65536, else SHOTKV_ERR_UNSUPPORTED_SHAPE (use the workspace form).
 *   - The first call on each device looks up the table's device address; make that first call
 *     outside any stream capture.
 *   - All calls on a device share the one table, and it keeps the previous call's contents: each
 *     call overwrites every entry it reads, but two calls that overlap on the GPU (different
 *     streams, or the same stream from two threads) race on it.  Serialise them.
 * All other arguments, outputs and return codes are those of shotkv_select_shots.  */
SHOTKV_API int shotkv_select_shots_static(shotkv_ctx* ctx, const shotkv_dims* dims,
                               const shotkv_policy* policy, const float* token_importance,
                               const int32_t* offsets_host, float* shot_scores, uint8_t* keep,
                               int32_t* kept_idx, int32_t* kept_count, int32_t Mcap, void* stream);

/* Compress (Section 5.1, Compress equation): gathers the kept rows of every KV head of a layer.
 *   Kc[b][l][g][j] = K[b][l][g][kept_idx[b][l][j]]  for j < kept_count[b][l]; same for V.
 *   K, V   device [B][L][Hkv][N][d] bf16     Kc, Vc  device [B][L][Hkv][Mcap][d] bf16
 * Rows j >= kept_count[b][l] of Kc/Vc are left untouched.  Bit-exact copy.  */
SHOTKV_API int shotkv_compact_kv(shotkv_ctx* ctx, const shotkv_dims* dims,
                      const shotkv_bf16* K, const shotkv_bf16* V,
                      const int32_t* kept_idx, const int32_t* kept_count, int32_t Mcap,
                      shotkv_bf16* Kc, shotkv_bf16* Vc, void* stream);

/* The whole of Phase 1 in one call: score, select, compact.  Without
 * SHOTKV_FLAG_TOKEN_IMPORTANCE the shot scores are formed directly from per-shot partial sums
 * (K is streamed once and per-token importance is never materialised; token_importance is
 * ignored and may be NULL); with it the call equals the three calls above in sequence.
 * When the units are very short (fewer than 16 tokens on average with more than 128 window rows
 * G*W, fewer than 40 otherwise) the call also goes through per-token importances, kept in the
 * workspace: the cost of that route does not grow with S.  Longer units -- with 256 window rows
 * that includes sentence-sized units and 16-token chunks -- stay on the single-pass form, whose
 * workspace grows with S (two floats per unit, window row and KV head).  Arguments as in those
 * calls.
 *   Units (b, l) are independent (Algorithm 1 compresses layer by layer), so the single-pass form
 *   can cut them into up to four groups -- whole prompts, or runs of layers when B = 1 -- and
 *   reduce, select and compact one group on a stream the context owns while `stream` works on the
 *   next (shotkv_set_pipeline_groups; by default only the host-buffer variant below does so).  To
 *   the caller everything still happens on `stream`: the work starts after what was enqueued there
 *   before the call, and what is enqueued there after the call starts once all of it has finished.
 *   Every unit's results are the same whatever the grouping, up to fp32 summation order.  */
SHOTKV_API int shotkv_prefill_compress(shotkv_ctx* ctx, const shotkv_dims* dims, const shotkv_policy* policy,
                            const shotkv_bf16* Qwin, const shotkv_bf16* K, const shotkv_bf16* V,
                            const int32_t* offsets_host,
                            float* shot_scores, uint8_t* keep, int32_t* kept_idx,
                            int32_t* kept_count, int32_t Mcap,
                            shotkv_bf16* Kc, shotkv_bf16* Vc,
                            float* token_importance, uint32_t flags,
                            void* ws, size_t ws_bytes, void* stream);

/* Same, for callers whose tensors live in HOST memory.  Copies Qwin and K to the device arena, runs
 * Phase 1 and delivers the results to the host buffers, all on `stream`; returns after
 * enqueueing.  Outputs with a NULL host pointer are not delivered.  On large inputs K goes up one
 * group of units at a time, each just ahead of its scoring pass, so that later uploads run beside
 * the gathers and write-backs of earlier groups.
 *   Page-locked buffers (cudaHostAlloc / cudaHostRegister) make the copies asynchronous, and
 *   more: V is only ever gathered (the Compress equation takes the kept tokens' rows), so a
 *   page-locked V_host is read in place by the compaction kernel -- only the kept rows cross the
 *   bus -- and page-locked Kc_host / Vc_host are written in place by it (rows at and beyond
 *   kept_count are then left untouched).  Pageable buffers are staged whole through the arena.
 *   arena  device buffer of >= shotkv_host_arena_bytes(dims, Mcap) bytes, 256-byte aligned
 * The host outputs are valid once `stream` has been synchronised.  */
SHOTKV_API size_t shotkv_host_arena_bytes(const shotkv_dims* dims, int32_t Mcap);
SHOTKV_API int shotkv_prefill_compress_host(shotkv_ctx* ctx, const shotkv_dims* dims,
                                 const shotkv_policy* policy,
                                 const shotkv_bf16* Qwin_host, const shotkv_bf16* K_host,
                                 const shotkv_bf16* V_host, const int32_t* offsets_host,
                                 float* shot_scores_host, uint8_t* keep_host,
                                 int32_t* kept_idx_host, int32_t* kept_count_host, int32_t Mcap,
                                 shotkv_bf16* Kc_host, shotkv_bf16* Vc_host,
                                 void* arena, size_t arena_bytes, void* stream);

/* ---- decode (Algorithm 1, Phase 2) --------------------------------------------------------- */

/* Decode-side cache of B sequences x L layers.  The caller allocates the device arrays and fills
 * the struct through shotkv_decode_init; the library updates T and n_dec on the host.  Every
 * sequence generates one token per step, so T and n_dec are the same for all (b, l).  */
typedef struct {
    shotkv_dims   dims;        /* B, L, H, Hkv, d are used                                         */
    shotkv_policy policy;      /* r_d, recompress_every are used                                   */
    int32_t Dcap;              /* rows per (b,l,g) of Kd/Vd; needs >= n_dec+1 at every step         */
    int32_t Mcap;              /* rows per (b,l,g) of the compressed prefill keys Kc                */
    int32_t T;                 /* tokens generated so far                                          */
    int32_t n_dec;             /* decode entries currently held per (b,l)                          */
    shotkv_bf16* Kd;           /* device [B][L][Hkv][Dcap][d]                                      */
    shotkv_bf16* Vd;           /* device [B][L][Hkv][Dcap][d]                                      */
    float*   acc;              /* device [B][L][Dcap]  accumulated Score_decoding per entry        */
    int32_t* born;             /* device [B][L][Dcap]  generation step (0-based) of each entry     */
    void*    ws;               /* device workspace, >= shotkv_decode_workspace_bytes()             */
    size_t   ws_bytes;
} shotkv_decode_state;

SHOTKV_API size_t shotkv_decode_workspace_bytes(const shotkv_dims* dims, int32_t Dcap);
/* Smallest Dcap that never overflows over `steps` steps under `policy`. */
SHOTKV_API int32_t shotkv_decode_capacity(const shotkv_policy* policy, int32_t steps);
/* Validates and fills `state` (T = n_dec = 0).  Touches no device memory.  */
SHOTKV_API int shotkv_decode_init(shotkv_ctx* ctx, const shotkv_dims* dims, const shotkv_policy* policy,
                       int32_t Dcap, int32_t Mcap, shotkv_bf16* Kd, shotkv_bf16* Vd, float* acc,
                       int32_t* born, void* ws, size_t ws_bytes, shotkv_decode_state* state);

/* One generation step for all (b, l) (decoding score equation and TopK rule of Section 5.1):
 *   1. append k_new/v_new as decode entry n_dec with score 0; T += 1;
 *   2. for every query head, softmax of q.k/sqrt(d) over the kept prefill keys Kc[..][0..M) and
 *      all decode keys together (M = kept_count[b][l]); acc[j] += sum over the H heads of the
 *      weight on decode entry j;
 *   3. if T % recompress_every == 0: keep the k = min(n_dec, floor(r_d*T)) entries greatest in
 *      (acc descending, index ascending), compacted in index order (Kd, Vd, acc, born).  With
 *      protect_recent = P > 0 the entries generated in the last P steps are kept first, whatever
 *      their score, and the others fill what is left of k (k is raised to P if it is smaller).
 *   q device [B][L][H][d] bf16;  k_new, v_new device [B][L][Hkv][d] bf16;
 *   Kc device [B][L][Hkv][Mcap][d] bf16;  kept_count device [B][L] i32.  */
SHOTKV_API int shotkv_decode_step(shotkv_ctx* ctx, shotkv_decode_state* state,
                       const shotkv_bf16* q, const shotkv_bf16* k_new, const shotkv_bf16* v_new,
                       const shotkv_bf16* Kc, const int32_t* kept_count, void* stream);

/* The same step with the attention output of the step fused in (Preliminary: attention over the
 * cached keys and values; Section 5.1: the decoding score is built from "the attention weight
 * from the current generation step", i.e. from weights a decode step computes anyway).  Besides
 * everything shotkv_decode_step does,
 *   attn_out[b][l][h][:] = sum_t alpha_{t,h} * v_t
 * over the kept prefill entries (Kc, Vc rows [0, M)) and all decode entries, the new token
 * included, with alpha the softmax weights of step 2 above; evaluated before the eviction of
 * step 3.  K and V are each read once; the scores cost no further pass over the cache.
 *   Vc device [B][L][Hkv][Mcap][d] bf16;  attn_out device [B][L][H][d] f32 (written in full).  */
SHOTKV_API int shotkv_decode_step_attend(shotkv_ctx* ctx, shotkv_decode_state* state,
                       const shotkv_bf16* q, const shotkv_bf16* k_new, const shotkv_bf16* v_new,
                       const shotkv_bf16* Kc, const shotkv_bf16* Vc, const int32_t* kept_count,
                       float* attn_out, void* stream);

/* The work partition the scoring pass uses for `dims` on a GPU with `sm_count` SMs (host only; a
 * diagnostic and test aid).  Every prompt's keys [0, N) are cut into pieces at the shot boundaries
 * (when offsets_host is given) and at the ends of `nchunk` equal chunks of `chunk_keys` keys (whole
 * 128-key tiles); per (piece, window row) the scoring kernel emits one softmax partial.
 *   pieces_out  host [B][cap][3] = (lo, hi, segment) per piece; segment 0 = before the first shot,
 *               i+1 = shot i, S+1 = the question, S+2 = list padding.  May be NULL.
 * Returns the number of pieces per prompt (<= S + 67), or a negative error.  */
SHOTKV_API int32_t shotkv_plan_pieces(const shotkv_dims* dims, const int32_t* offsets_host, int32_t sm_count,
                           int32_t* nchunk, int32_t* chunk_keys, int32_t* pieces_out, int32_t cap);

/* ---- instrumentation (used by the benchmark; not part of the method) ------------------------ */

/* How the window logits are exponentiated in the scoring pass (the alpha of the prefill score
 * equation, Section 5.1).  Both modes compute the same softmax sums; they differ in how the
 * reference exponent of a window row is chosen.
 *   SHOTKV_SCORING_FAST (default): per work item the reference is fixed from the item's first
 *     128 keys and sums are carried in fp32 with about 2^158 of headroom above it; any item
 *     whose sums leave that range is recomputed on the device by the exact kernel, in the same
 *     call, so the outputs are those of the exact mode up to fp32 rounding.
 *   SHOTKV_SCORING_EXACT: every item runs the exact kernel (a running maximum per row).
 * Takes effect for the calls that follow on this context.  */
#define SHOTKV_SCORING_FAST 0
#define SHOTKV_SCORING_EXACT 1
SHOTKV_API int shotkv_set_scoring_mode(shotkv_ctx* ctx, int mode);
/* Work items (a run of a unit's keys) that the exact kernel recomputed after the fast one, summed
 * over the calls finished so far on this context.  A diagnostic: 0 on ordinary inputs.  */
SHOTKV_API uint64_t shotkv_repaired_items(const shotkv_ctx* ctx);

/* Failure detection.  The tensor-core kernels of this library (the scoring pass of Section 5.1's
 * prefill score equation and the per-token second pass) hand tiles between warps through shared-
 * memory barriers.  Every such wait is bounded: after `cycles` SM clock cycles (default 4e9, about
 * two seconds) the waiting warp gives up, raises its CTA's abort flag and a host-visible error
 * word, all roles leave their loops, copies in flight are waited for (bounded again), tensor
 * memory is released and the kernel returns.  The next call on the context then returns
 * SHOTKV_ERR_TIMEOUT once (the outputs of the call that gave up are invalid); the call after
 * that proceeds normally.  shotkv_set_wait_limit changes the limit for later launches of this
 * context (0 restores the default).  */
SHOTKV_API int shotkv_set_wait_limit(shotkv_ctx* ctx, int64_t cycles);
/* Runs the bounded-wait helpers on purpose into their limit, so that the give-up path can be
 * checked on any installation without disturbing a real kernel: one CTA, two barriers nobody
 * arrives on.  Warp 0 waits as the epilogue warps do, with `limit_cycles` (1e3..1e9); one thread
 * of warp 1 waits as the producer and MMA threads do, with four times that, and must leave early
 * because warp 0 raised the abort flag.  Tensor memory is allocated and released around it as in
 * the kernels' exit path.  Nothing faults and nothing spins past its limit.
 *   report host [4] = {warp 0's wait succeeded (0 expected), warp 1's wait succeeded (0 expected),
 *                      abort flag at exit (1 expected), cycles warp 1 waited (< 4*limit_cycles)}
 * This call SYNCHRONISES `stream`.  It leaves the error word raised exactly as a real give-up
 * does: the next call on the context returns SHOTKV_ERR_TIMEOUT, the one after that succeeds.  */
SHOTKV_API int shotkv_selftest_bounded_wait(shotkv_ctx* ctx, int64_t limit_cycles, int32_t* report /* [4] */,
                                            void* stream);

/* SM cycles and nanoseconds that the first CTA of the most recent scoring launch of this context
 * ran for (its own cycle counter and the GPU's nanosecond timer, read at its start and end).  Their
 * quotient is the SM clock the kernel really ran at -- under a power cap that is not the clock a
 * sampler reads between kernels -- and cycles / tiles per SM is the kernel's cost per tile in the
 * unit its arithmetic is counted in.  Valid once the launch has finished (synchronise first).  */
SHOTKV_API int shotkv_last_scoring_clock(const shotkv_ctx* ctx, int64_t* cycles, int64_t* nanoseconds);

/* Groups the single-pass form of shotkv_prefill_compress pipelines its units in: 0 (default)
 * chooses -- one group for device buffers, one per 256 MB of K (at most 4) for the host-buffer
 * variant, where the groups overlap uploads with write-backs --, 1 runs every step on the
 * caller's stream, 2..4 force that many groups where there are enough prompts (or layers).  A
 * tuning and testing knob; the paper has no counterpart.  */
SHOTKV_API int shotkv_set_pipeline_groups(shotkv_ctx* ctx, int groups);

/* When enabled, shotkv_prefill_compress (single-pass form) and shotkv_decode_step record CUDA
 * events on their stream at their stage boundaries; the last 64 calls are retained.  */
SHOTKV_API int shotkv_profile_enable(shotkv_ctx* ctx, int enable);
/* Stage durations in milliseconds of the profiled call made `calls_back` calls ago (0 = latest);
 * waits for that call to finish.  Prefill: {scoring kernel, per-shot reduce, select, compact},
 * each summed over the groups of a pipelined call (stages of different groups overlap, so the
 * sum can exceed the call's duration); decode: {score kernel, accumulate+evict, -1, -1}.  Returns the number of stages or a negative
 * error. */
SHOTKV_API int shotkv_profile_read(shotkv_ctx* ctx, int calls_back, float* stage_ms /* [4] */);
/* Kernels launched through this context since it was created. */
SHOTKV_API uint64_t shotkv_launch_count(const shotkv_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* SHOTKV_H_ */
