/*
 * dkv.h -- C ABI of libdkv: DynamicKV prefill-time KV-cache compression on one NVIDIA B200.
 *
 * The library implements the data-parallel path of Algorithm 1 ("DynamicKV in Prefill Phase",
 * arXiv 2412.14838): per layer, score every prefix token against the observation-window
 * queries (Eq. 1-2), keep the per-layer maximum budget B^l per head (Eq. 3), every m layers
 * re-derive the per-layer counts from a global top-K over all accumulated scores (Eq. 4-6),
 * and shrink the buffers of all preceding layers to those counts.
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, 16-byte aligned, contiguous in
 *     the stated layout, unless the argument is documented as a host pointer.  The library never
 *     frees or reallocates caller memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls enqueue
 *     work and return; only dkv_create, dkv_destroy, dkv_get_counts, dkv_last_status and
 *     dkv_run_prefill_pass_host synchronise.
 *   - A context belongs to one device (the one current at dkv_create) and to one stream at a time.
 *   - Return value: 0 = DKV_OK, negative = error (below).  Nothing is printed, nothing aborts.
 *   - Layer numbers are 0-based.  Algorithm 1's test "l % m == 0" uses 1-based l, i.e. an update
 *     follows API layers m-1, 2m-1, ...
 *   - Shapes: L layers, Hq query heads, Hkv KV heads (G = Hq/Hkv), D head size, Bt samples, S prompt
 *     length including the window, ws window, P = S - ws prefix tokens, N = wt - ws average budget,
 *     Bl = B^l = N * r_max per-layer maximum, Bl' = min(Bl, P).
 *   - bf16 tensors are raw 16-bit patterns.  Samples of a batch are independent problems.
 */
#ifndef DKV_H_
#define DKV_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DKV_OK                 0
#define DKV_ERR_INVALID_ARG   -1   /* NULL/misaligned pointer, value out of range                  */
#define DKV_ERR_STATE         -2   /* call order: e.g. select before score                         */
#define DKV_ERR_CUDA          -3   /* a CUDA runtime call failed (dkv_last_cuda_error has the code) */
#define DKV_ERR_TIMEOUT       -4   /* a bounded device-side wait ran out                           */
#define DKV_ERR_UNSUPPORTED   -5   /* shape outside the compiled set                               */
#define DKV_ERR_NOMEM         -6   /* device or host allocation failed                             */
#define DKV_ERR_TOO_LARGE     -7   /* dkv_score_static: the problem does not fit the static scratch */

#define DKV_MAX_LAYERS        128
#define DKV_MAX_LAYER_BUDGET  16384  /* Bl  */
#define DKV_MAX_WINDOW_ROWS   256    /* ws * G */

/* Alternative readings of passages where the paper is silent or inconsistent (dkv_config.flags).
 * With all bits clear the library computes the default readings.                                  */
#define DKV_F_WINDOW_MEAN  0x1u  /* Algorithm 1's scoring line takes the MEAN over the window rows (and the
                                    query heads of a group) where Eq. 2 is read as a sum: scores / (ws*G)  */
#define DKV_F_PRORATA      0x2u  /* Eq. 6 at an update after l < L layers uses the budget of those layers,
                                    B = (wt-ws)*l, instead of (wt-ws)*L                                    */
#define DKV_F_NORM_MINMAX  0x4u  /* Update_Buffer_Length's "Norm ... range in (0,1)" is min-max scaling:
                                    t_i = (cnt_i - min)/(max - min), all 1 if every layer counts the same  */
#define DKV_F_ALL          0x7u

typedef struct dkv_ctx dkv_ctx;     /* opaque; owns score history, kept indices, ranks, counts, workspace */

/* Problem statement of Algorithm 1 (its inputs r_max, m, wt, ws, S, d_k) plus the model shape. */
typedef struct {
  int32_t n_layers;         /* L   : 1..DKV_MAX_LAYERS                                            */
  int32_t n_q_heads;        /* Hq  : multiple of n_kv_heads                                       */
  int32_t n_kv_heads;       /* Hkv                                                                */
  int32_t head_dim;         /* D   : 64 or 128                                                    */
  int32_t batch;            /* Bt                                                                 */
  int32_t seq_len;          /* S   : includes the window; S > ws                                  */
  int32_t window;           /* ws  : ws * G <= DKV_MAX_WINDOW_ROWS                                */
  int32_t pool_kernel;      /* odd width of the 1-D pooling of Eq. 2, 1..255                      */
  int32_t pool_kind;        /* 0 = max-pool (default), 1 = average over the neighbours that exist */
  int32_t avg_budget;       /* N = wt - ws : retained prefix tokens per head per layer on average */
  int32_t layer_max;        /* Bl = floor(N * r_max), N <= Bl <= DKV_MAX_LAYER_BUDGET             */
  int32_t update_interval;  /* m >= 1                                                             */
  uint32_t flags;           /* DKV_F_* bits, 0 = the default readings                             */
} dkv_config;

/* Create a context for `cfg` on the current device (host call; allocates device memory:
 * score history 4*L*Bt*Hkv*P bytes, kept indices and ranks 8*L*Bt*Hkv*Bl' bytes, small workspaces).
 * Errors: INVALID_ARG, UNSUPPORTED, NOMEM, CUDA.  On error *out is NULL. */
int dkv_create(const dkv_config* cfg, dkv_ctx** out);
/* Free everything the context owns (synchronises the device). */
int dkv_destroy(dkv_ctx* ctx);
/* Forget all layers: a new prompt.  Enqueued on `stream`. */
int dkv_reset(dkv_ctx* ctx, void* stream);

/* (1) Eq. 1-2 / Algorithm 1 scoring line.  For every sample b, KV head h and prefix position j < P:
 *       raw[j]   = sum over the G query heads of the group and the ws window rows r of
 *                  softmax_row(q . K^T / sqrt(D))[j], row r's softmax running over keys 0 .. P+r;
 *       score[j] = max of raw over |j' - j| <= pool_kernel/2, 0 <= j' < P.
 *     q_win : bf16 [Bt, Hq, ws, D]   queries of the last ws positions
 *     k     : bf16 [Bt, Hkv, S, D]   keys of the layer
 *     scores_out : fp32 [Bt, Hkv, P] optional copy of the result (NULL = keep it in the context only)
 *     bf16 inputs, fp32 accumulation.  Stores the scores as layer `layer` of the context's history. */
int dkv_score(dkv_ctx* ctx, int32_t layer, const void* q_win, const void* k, float* scores_out, void* stream);

/* Scoring for callers that cannot allocate device memory.  (The paper has no counterpart: this is a
 * packaging of step (1) above, not a step of the method.)
 *
 * Who needs it: programs that must not reach cudaMalloc on this path.  Typical cases are an inference
 * server that has handed all of the GPU's memory to its own pool, so that a library-side cudaMalloc
 * would simply fail, and a request path on which cudaMalloc's device-wide synchronisation would stall
 * every other stream.  dkv_create allocates (history, indices, workspaces), so such callers cannot own
 * a context; this call needs none.  It calls neither cudaMalloc nor cudaFree nor any allocating
 * library routine.
 *
 * What it does: exactly dkv_score's computation for one layer, same kernels, writing the pooled
 * scores fp32 [Bt, Hkv, P] to scores_out (required).  Only the scoring fields of cfg are used
 * (heads, head_dim, batch, seq_len, window, pool_kernel); the whole cfg must still be valid.
 * Its scratch (partial softmax statistics of sweep 1, plus status words) is a fixed array of
 * DKV_STATIC_SCRATCH_BYTES inside the library image: every GPU that loads libdkv holds those bytes
 * until the process exits.  A problem that needs more returns DKV_ERR_TOO_LARGE and launches nothing;
 * the need is 256 + Bt*Hkv * slots * 2048 bytes with slots about (SM count)/(Bt*Hkv) + 2, i.e. some
 * 0.3 MB for 8 heads and 2 MB for 512 heads on a 148-SM part.
 *
 * The first call on each device looks up the array's device address and sets the kernels' shared
 * memory attribute (host-side, once).  Make that first call before starting any stream capture, and
 * before the caller's own pool takes the rest of the device memory: with CUDA's default lazy module
 * loading the library image, and with it this array, is placed on the device at the first use of one of
 * its kernels or symbols, i.e. inside that first call (CUDA_MODULE_LOADING=EAGER moves it to load time).
 * A wait inside the kernels that runs out (see dkv_last_status) is reported by dkv_static_last_status.
 * All calls on a device share the one array, and it keeps whatever the last call left: the call
 * clears the status words it needs zeroed and overwrites every statistic before reading it, so
 * calls that follow one another on a stream are independent.  Calls that can overlap on the GPU
 * (different streams, different host threads) race on the array: serialise them.
 * q_win : bf16 [Bt, Hq, ws, D];  k : bf16 [Bt, Hkv, S, D];  device pointers, 16-byte aligned. */
#define DKV_STATIC_SCRATCH_BYTES (4u << 20)
int dkv_score_static(const dkv_config* cfg, const void* q_win, const void* k, float* scores_out, void* stream);

/* (1') Eq. 2 with Eq. 1's denominators given.  A prefill attention kernel that has just run over the prompt
 * already holds, for every query row, the logarithm of its softmax denominator (the "log-sum-exp" such
 * kernels return beside their output).  With those values for the ws window rows the scores of step (1)
 * need one sweep over the keys instead of two:
 *       raw[j] = sum over the group's G query heads and the ws window rows r of exp(q . k_j / sqrt(D) - lse[.., r]),
 * pooled as in step (1).  The result equals dkv_score's when
 *       lse[b, hq, r] = ln( sum over keys i <= P + r of exp(q[b,hq,r] . k[b,hq/G,i] / sqrt(D)) )   (natural log).
 *     lse : fp32 [Bt, Hq, ws], device, 4-byte aligned; finite.  Other arguments as for dkv_score.
 * The library does not check lse against k: a wrong normaliser scales that row's contribution. */
int dkv_score_lse(dkv_ctx* ctx, int32_t layer, const void* q_win, const void* k, const float* lse,
                  float* scores_out, void* stream);

/* Store caller-computed scores fp32 [Bt, Hkv, P] (finite, >= 0) as layer `layer` of the history,
 * in place of dkv_score (e.g. scores emitted by a fused prefill attention kernel). */
int dkv_set_scores(dkv_ctx* ctx, int32_t layer, const float* scores, void* stream);

/* (2) Eq. 3 / Algorithm 1 "topk(B^l)".  Per (b, h): the Bl' positions with the largest score under the
 *     total order (score descending, position ascending).  The context keeps them in that order, which
 *     is the order Algorithm 1's topk() yields and the order of the buffer rows dkv_compact writes.
 *     idx_out  : int32 [Bt, Hkv, Bl'] the kept positions, ascending (optional)
 *     rank_out : int32 [Bt, Hkv, Bl'] place of each of those in the total order, 0 = best, i.e. its
 *                buffer row (optional)
 *     Sets count[b][layer] = Bl'.  Needs the layer's scores (else DKV_ERR_STATE).  Also files the head's
 *     scores by their leading bits for the later global top-K of dkv_rebudget. */
int dkv_select_topk(dkv_ctx* ctx, int32_t layer, int32_t* idx_out, int32_t* rank_out, void* stream);

/* (3) Eq. 4-6 / Update_Buffer_Length after `upto_layer` layers (1..L; all of them scored and selected).
 *     Per sample: k = min(N*Hkv*l, l*Hkv*P) largest history scores of layers [0, l), ties to the lowest
 *     flat index (layer, head, position); cnt_i = hits in layer i; Z_i = floor(Bl*cnt_i / max cnt);
 *     Z'_i = floor(Z_i * N*L / sum Z); count[b][i] = min(count[b][i], Z'_i).  All on the device.
 *     counts_out : int32 [Bt, L] device copy of the counts after the update (optional). */
int dkv_rebudget(dkv_ctx* ctx, int32_t upto_layer, int32_t* counts_out, void* stream);

/* (4) Algorithm 1's buffer build and truncation for one layer.  Buffer rows are in Algorithm 1's own
 *     order: row r of a head holds its r-th best position (score descending, ties by position), so
 *     that truncating to a smaller count keeps a prefix; the ws window rows follow the kept rows.
 *     k_src, v_src != NULL : gather.  kb[b,h,r] = k_src[b,h,pos_r] for r < c, kb[b,h,c:c+ws] = k_src[b,h,P:S],
 *                            same for v; c = count[b][layer].  k_src, v_src : bf16 [Bt, Hkv, S, D].
 *     k_src == v_src == NULL : shrink kb/vb in place to the current count c: rows [0, c) stay, the window
 *                            rows move up behind them.
 *     kb, vb  : bf16 [Bt, Hkv, Bl' + ws, D] fixed stride; rows past the valid length are unspecified.
 *     len_out : int32 [Bt, Hkv] valid rows including the window (optional). */
int dkv_compact(dkv_ctx* ctx, int32_t layer, const void* k_src, const void* v_src, void* kb, void* vb,
                int32_t* len_out, void* stream);

/* Shrink (as above) the buffers of all layers [0, upto_layer) in one launch.
 * kb, vb : HOST arrays of upto_layer device pointers. */
int dkv_compact_all(dkv_ctx* ctx, int32_t upto_layer, void* const* kb, void* const* vb, void* stream);

/* Algorithm 1's loop over all L layers: score, select, gather each layer; after every m-th layer (and
 * after the last one if L % m != 0) rebudget and shrink all preceding layers.  Resets the context first.
 * q_win, k, v, kb, vb : HOST arrays of L device pointers (layouts as above).
 * All layers' tensors must be resident when the call is made: the scoring kernel is launched once per group of
 * consecutive layers (sweep 2 of one group, sweep 1 of the next), the steps that consume a layer's scores run
 * beside the following groups' scoring.  The results are those of the layer-by-layer loop.
 * The first call with a given set of pointers records the whole pass as a CUDA graph (on an internal stream
 * that forks from `stream` and rejoins it); later calls with the same pointers replay it, whatever the
 * buffers then contain.  The plain sequence of launches is used instead while dkv_profile is on, when
 * `stream` is itself being captured, or if the capture fails. */
int dkv_run_prefill_pass(dkv_ctx* ctx, const void* const* q_win, const void* const* k, const void* const* v,
                         void* const* kb, void* const* vb, void* stream);

/* Algorithm 1's loop when the caller's prefill attention kernel has already produced, for every layer, the
 * log-denominators of the window rows (see dkv_score_lse): every layer is scored in one sweep over its keys.
 * lse : HOST array of L device pointers, each fp32 [Bt, Hq, ws] (natural logarithm), 4-byte aligned.
 * Everything else as dkv_run_prefill_pass, including the recording of the pass as a CUDA graph.  (Section 4.3
 * notes that the scoring needs the window rows' attention probabilities explicitly, which a fused attention
 * kernel does not return; its log-denominators are what it does return.) */
int dkv_run_prefill_pass_lse(dkv_ctx* ctx, const void* const* q_win, const void* const* k, const void* const* v,
                             const float* const* lse, void* const* kb, void* const* vb, void* stream);

/* The same pass with all tensors in HOST memory (pinned memory recommended): each layer's q and k
 * are copied to device staging buffers owned by the context and processed; of v only the kept rows are
 * needed (Algorithm 1 gathers V_c at the selected indices), so where v[l] is page-locked memory that
 * kernels can address (cudaHostAlloc / cudaHostRegister) the gather reads those rows in place and the
 * rest of v never crosses the bus; pageable v is copied in full like k.  After the last update
 * the counts and, of every layer's kb/vb, the valid rows of every head (count + ws; the rest of the
 * fixed-stride host buffers is left untouched) are copied back.  Synchronises.
 * q_win, k, v, kb, vb : host arrays of L HOST pointers; counts_out : host int32 [Bt, L]. */
int dkv_run_prefill_pass_host(dkv_ctx* ctx, const void* const* q_win, const void* const* k,
                              const void* const* v, void* const* kb, void* const* vb, int32_t* counts_out);

/* Bytes the last dkv_run_prefill_pass_host of this context moved: host to device (q, k, and v in full or
 * its gathered rows) and device to host (counts and the valid rows of kb/vb).  h2d, d2h : host int64. */
int dkv_host_pass_bytes(dkv_ctx* ctx, int64_t* h2d, int64_t* d2h);

/* Fixed-pattern budgets: the per-layer schedules of the methods the paper compares with (Section 5.1,
 * "Baselines"), applied through the same select / compact kernels in place of Eq. 4-6.  Needs every layer
 * selected.  count[b][i] = min(count[b][i], schedule_i) on the device; follow with dkv_compact_all (layers
 * gathered later pick the new count up by themselves).
 *   DKV_POLICY_UNIFORM : schedule_i = N in every layer (a fixed per-layer cache, as SnapKV-like methods keep).
 *   DKV_POLICY_PYRAMID : schedule_i = N + floor(N (L-1-2i) / (2 (L-1))), falling linearly with depth from about
 *                        3N/2 to N/2 (the pyramid pattern), summing to N*L up to the floors; N when L = 1.
 *   counts_out : int32 [Bt, L] device copy of the counts after the call (optional). */
#define DKV_POLICY_UNIFORM 0
#define DKV_POLICY_PYRAMID 1
int dkv_apply_policy(dkv_ctx* ctx, int32_t policy, int32_t* counts_out, void* stream);
/* Selection by position, without scores, in place of dkv_select_topk for one layer: every head keeps the first
 * n_sink and the last n_recent of its P prefix positions (attention sinks plus a window of the most recent
 * tokens, as StreamingLLM-like methods keep), ascending, each once if the two ranges meet.  The kept number must
 * not exceed Bl'.  Sets count[b][layer]; dkv_compact then gathers those rows.  Such a layer has no place in the
 * global top-K: dkv_rebudget over it returns DKV_ERR_STATE. */
int dkv_select_positions(dkv_ctx* ctx, int32_t layer, int32_t n_sink, int32_t n_recent, void* stream);

/* Decoding over the compressed cache (Section 4.3: decoding is the model's own attention, Eq. 1, over what
 * the prefill phase kept).  For layers [layer0, layer0 + n_layers), every sample b, query head hq and each of
 * the nq new queries:  out = softmax(q . Kb^T / sqrt(D)) Vb  over the rows [0, count[b][layer] + ws) of KV head
 * hq / G's buffers, the lengths being read from the context's device-side counts (they differ per layer).
 * The nq queries of a sample are independent: each sees the whole compressed cache.
 *   q_dec : HOST array of n_layers device pointers, bf16 [Bt, Hq, nq, D];  nq >= 1, G * nq <= 64
 *   kb, vb: HOST arrays of n_layers device pointers, the buffers dkv_compact wrote (layers must be gathered)
 *   out   : HOST array of n_layers device pointers, fp32 [Bt, Hq, nq, D]
 * bf16 inputs, fp32 accumulation.  One launch covers up to 64 layers; partial results of the thread blocks
 * that share a head go through a scratch array the context allocates on first use (and enlarges when a call
 * needs more; that one call synchronises the device). */
int dkv_decode_attend(dkv_ctx* ctx, int32_t layer0, int32_t n_layers, int32_t nq, const void* const* q_dec,
                      const void* const* kb, const void* const* vb, float* const* out, void* stream);

/* Copy the current counts to host int32 [Bt, L] (synchronises `stream`). */
int dkv_get_counts(dkv_ctx* ctx, int32_t* host_counts, void* stream);
/* Device-side views for inspection, owned by the context: the history scores of a layer
 * (fp32 [Bt,Hkv,P]) and the positions it currently keeps, in buffer order (int32 [Bt,Hkv,Bl'], the
 * first held[b][layer] entries of each head valid; entry r is the position of buffer row r).
 * Either out pointer may be NULL. */
int dkv_layer_views(dkv_ctx* ctx, int32_t layer, const float** scores, const int32_t** idx);
/* The positions a gathered layer currently keeps, ascending: sorted_out int32 [Bt,Hkv,Bl'], device,
 * the first held[b][layer] entries of each head written. */
int dkv_kept_sorted(dkv_ctx* ctx, int32_t layer, int32_t* sorted_out, void* stream);
/* Device-side views of the last update's intermediate integers, int32 [Bt, L] each:
 * cnt (Eq. 4 hits per layer), Z (Eq. 5), Zp (Eq. 6), and held (rows each layer's buffers hold now). */
int dkv_budget_views(dkv_ctx* ctx, const int32_t** cnt, const int32_t** z, const int32_t** zp, const int32_t** held);
/* Convenience for inspecting the views above: copy `bytes` from device memory to host memory and
 * synchronise `stream`. */
int dkv_memcpy_to_host(dkv_ctx* ctx, void* host_dst, const void* dev_src, uint64_t bytes, void* stream);
/* Copy the status words to host int32 [8] (synchronises the device):
 * [0] first device-side failure since the last report (0 = none; else the number, 101..107, of the wait in
 *     the scoring kernel that ran out first), [1] kernels launched since dkv_create (host counter),
 * [2] the thread block of that wait.
 * Returns DKV_OK when [0] is 0, else DKV_ERR_TIMEOUT: some wait inside a scoring launch since the last
 * report gave up, and the scores of the layers scored since then are not to be used.  The kernel itself
 * ended normally (no trap; its copies drained, its tensor memory freed), the context stays usable, and the
 * failure is reported once: the device words are cleared by the call that reports it. */
int dkv_last_status(dkv_ctx* ctx, int32_t* host_status);
/* The same for dkv_score_static, whose status words live in the library's static scratch: host int32 [8] as
 * above ([1] is 0).  Synchronises the current device; DKV_OK or DKV_ERR_TIMEOUT.  The next dkv_score_static
 * call clears the words. */
int dkv_static_last_status(int32_t* host_status);
/* Limit of every wait inside the scoring kernel, in SM clock ticks (default 4e9, about 2 s; at least 1000).
 * A wait that runs out makes its thread block stop issuing work, finish, and record the failure for
 * dkv_last_status.  Applies to launches made after the call. */
int dkv_set_wait_limit(dkv_ctx* ctx, int64_t clock_ticks);
/* Test hook for the path above: in the launches that follow, thread block 0 never loads its key tile number
 * `tile` (0-based, per launch) of scoring sweep `sweep` (1 = statistics, 2 = emit), so the wait for that
 * tile runs out after the wait limit.  tile < 0 switches the hook off.  Nothing else is disturbed: no
 * invalid address, no trap. */
int dkv_debug_withhold_tile(dkv_ctx* ctx, int32_t sweep, int32_t tile);
/* Optional per-step timing.  While enabled, every step's launches are bracketed by a pair of CUDA
 * events on the step's stream.  dkv_profile_read synchronises the device and returns, per step
 * (DKV_STEP_*), the summed event time in milliseconds and the number of kernels covered since the
 * last read, then clears the sums.  ms, launches : host arrays of DKV_N_STEPS entries. */
#define DKV_STEP_SCORE_STATS 0   /* sweep 1 of the scoring: softmax statistics per window row */
#define DKV_STEP_SCORE_EMIT  1   /* sweep 2 of the scoring: per-token sums, pooled             */
#define DKV_STEP_SELECT      2
#define DKV_STEP_GATHER      3
#define DKV_STEP_REBUDGET    4
#define DKV_STEP_SHRINK      5
#define DKV_STEP_DECODE      6
#define DKV_N_STEPS          8
int dkv_profile(dkv_ctx* ctx, int enable);
int dkv_profile_read(dkv_ctx* ctx, double* ms, int64_t* launches);
/* Kernels this context has launched since dkv_create (host counter, no synchronisation); -1 if ctx is NULL. */
int64_t dkv_launch_count(dkv_ctx* ctx);
/* CUDA error code of the last DKV_ERR_CUDA on this context (0 = none). */
int dkv_last_cuda_error(dkv_ctx* ctx);
const char* dkv_strerror(int code);
/* Library version, 1000*major + minor. */
int dkv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DKV_H_ */
