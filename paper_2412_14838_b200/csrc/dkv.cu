// libdkv: context, argument checking and the C ABI declared in include/dkv.h.
// The method's steps (Algorithm 1 of arXiv 2412.14838) live in the kernel headers included here.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/dkv.h"
#include "common.cuh"
#include "compact.cuh"
#include "decode.cuh"
#include "rebudget.cuh"
#include "score_tc.cuh"
#include "select.cuh"

using namespace dkv;

struct ProfRec { cudaEvent_t a, b; int step; int launches; };

constexpr int kSideStreams = 4;
constexpr int kSelMaxSmem = DKV_MAX_LAYER_BUDGET * 8 + DKV_MAX_LAYER_BUDGET * 4;

struct dkv_ctx {
  dkv_config cfg;
  Shape s;
  int device;
  // device state
  float* d_scores;      // [L][Bt][Hkv][P]  pooled scores, the history A^b
  int* d_idx;           // [L][Bt][Hkv][Blc] kept positions, ascending
  int* d_count;         // [Bt][L] budget of each layer
  int* d_held;          // [Bt][L] rows the layer's buffers hold
  int* d_dbg;           // 3 x [Bt][L] : cnt, Z, Z' of the last update
  unsigned int* d_layer_hist; // [L][Bt][2048] first-digit histogram of every layer's scores (all heads of a sample)
  uint2* d_cand;              // [Bt][L*Hkv*P] (score bits, layer) of the scores in the global top-K's first bucket
  unsigned int* d_cand_n;     // [Bt]
  RbState* d_rb_state;        // [Bt]
  unsigned int* d_rb_above;   // [Bt][L]
  unsigned int* d_rb_hist1;   // [Bt][2048]
  unsigned int* d_rb_above2;  // [Bt][L]
  unsigned int* d_rb_hist2;   // [Bt][L][1024]
  int* d_status;        // [8]
  int sort_n;
  bool sel_reg;         // a head's scores fit the select kernel's registers and shared memory
  size_t sel_smem;
  // tensor-core scoring
  int n_sms, tc_grid, tc_slots;
  int pass_taper;       // group sizes halve towards the end of the pass
  int pass_group;       // layers per scoring launch of dkv_run_prefill_pass (1..tc::kMaxGroup)
  bool emit_backward;   // sweep 2 walks every CTA's slice from the end to the start
  bool host_v_staged;   // dkv_run_prefill_pass_host copies V in full even where the gather could read its rows in place
  long long host_h2d, host_d2h;   // bytes the last dkv_run_prefill_pass_host moved in either direction
  int retain_mb;        // MB of a sweep-1 job's keys (the end of every CTA's slice) marked to stay in L2 for sweep 2
  long long wait_cycles;   // limit of the scoring kernel's mbarrier waits (dkv_set_wait_limit)
  int withhold_sweep, withhold_tile;   // test hook of dkv_debug_withhold_tile (-1: off)
  float2* d_tc_stats;   // [3][kMaxGroup*Bt*Hkv][tc_slots][256]: partial softmax statistics, three jobs in rotation
  cudaStream_t hi;      // scoring launches of dkv_run_prefill_pass: highest priority, so that a freed SM goes to a
                        // waiting scoring CTA before the side streams' many short CTAs
  cudaStream_t upd;     // budget updates (rebudget + shrink) of dkv_run_prefill_pass, off the select streams
  cudaStream_t side[kSideStreams]; // side streams of dkv_run_prefill_pass (select / gather), layers in rotation
  int n_side;           // how many of them the pass uses
  cudaEvent_t ev_fork, ev_join[kSideStreams + 1], ev_update, ev_scored[DKV_MAX_LAYERS], ev_picked[DKV_MAX_LAYERS], ev_selected[DKV_MAX_LAYERS];
  // host state
  uint8_t scored[DKV_MAX_LAYERS], gathered[DKV_MAX_LAYERS], stale[DKV_MAX_LAYERS];
  uint8_t selected[DKV_MAX_LAYERS];     // 1: by scores (dkv_select_topk), 2: by position (dkv_select_positions)
  int sel_n[DKV_MAX_LAYERS];            // positions selected per head: Blc, or what dkv_select_positions kept
  // decoding over the compressed cache (allocated on first use, grown on demand)
  float* d_dec_scratch;
  size_t dec_scratch_floats;
  unsigned int* d_dec_tickets;          // [L][Bt*Hkv], zero between launches
  long long launches;
  // dkv_run_prefill_pass as a CUDA graph: captured on the first call with a set of pointers, replayed afterwards
  bool use_graph;
  cudaStream_t gstream;        // the graph is captured and replayed here, forked from / joined to the caller's stream
  cudaEvent_t ev_gfork, ev_gjoin;
  cudaGraphExec_t pass_exec;
  std::vector<const void*>* pass_key;
  long long pass_launches;
  int last_cuda;
  // optional per-step timing with CUDA events (dkv_profile)
  bool prof_on;
  std::vector<ProfRec>* prof_recs;
  size_t prof_used;
  double prof_ms[DKV_N_STEPS];
  long long prof_launches[DKV_N_STEPS];
  // staging for the host-buffer pass (allocated on first use)
  bool staged;
  void *st_q[2], *st_k[2], *st_v[2];
  void *st_kb[DKV_MAX_LAYERS], *st_vb[DKV_MAX_LAYERS];
  cudaStream_t st_copy, st_comp;
  cudaEvent_t ev_copied[2], ev_consumed[2];
};

namespace {

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int cuda_fail(dkv_ctx* c, cudaError_t e) {
  if (c) c->last_cuda = (int)e;
  return e == cudaErrorMemoryAllocation ? DKV_ERR_NOMEM : DKV_ERR_CUDA;
}
#define DKV_CUDA(ctx, call)                                   \
  do {                                                        \
    cudaError_t e__ = (call);                                 \
    if (e__ != cudaSuccess) return cuda_fail((ctx), e__);     \
  } while (0)
// After a launch: a launch error is reported once and cleared (cudaGetLastError), so that a refused launch
// does not make every later call of every context fail.
#define DKV_LAUNCHED(ctx)                                     \
  do {                                                        \
    (ctx)->launches++;                                        \
    cudaError_t e__ = cudaGetLastError();                     \
    if (e__ != cudaSuccess) return cuda_fail((ctx), e__);     \
  } while (0)

// Event pair around one step's launches; read back by dkv_profile_read.
struct ProfScope {
  dkv_ctx* c; cudaStream_t st; ProfRec* r;
  ProfScope(dkv_ctx* c_, int step, int launches, cudaStream_t st_) : c(c_), st(st_), r(nullptr) {
    if (!c->prof_on) return;
    if (c->prof_used == c->prof_recs->size()) {
      ProfRec n; n.step = 0; n.launches = 0;
      if (cudaEventCreate(&n.a) != cudaSuccess || cudaEventCreate(&n.b) != cudaSuccess) return;
      c->prof_recs->push_back(n);
    }
    r = &(*c->prof_recs)[c->prof_used++];
    r->step = step; r->launches = launches;
    cudaEventRecord(r->a, st);
  }
  ~ProfScope() { if (r) cudaEventRecord(r->b, st); }
};

size_t layer_scores(const Shape& s) { return (size_t)s.Bt * s.Hkv * s.P; }
size_t layer_idx(const Shape& s) { return (size_t)s.Bt * s.Hkv * s.Blc; }
size_t layer_kv_bytes(const Shape& s) { return (size_t)s.Bt * s.Hkv * s.S * s.D * 2; }
size_t layer_q_bytes(const Shape& s) { return (size_t)s.Bt * s.Hq * s.ws * s.D * 2; }
size_t layer_buf_bytes(const Shape& s) { return (size_t)s.Bt * s.Hkv * s.rows * s.D * 2; }

int validate(const dkv_config* c) {
  if (!c) return DKV_ERR_INVALID_ARG;
  if (c->n_layers < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->batch < 1) return DKV_ERR_INVALID_ARG;
  if (c->n_q_heads % c->n_kv_heads != 0) return DKV_ERR_INVALID_ARG;
  if (c->window < 1 || c->seq_len <= c->window) return DKV_ERR_INVALID_ARG;
  if (c->pool_kernel < 1 || c->pool_kernel % 2 == 0) return DKV_ERR_INVALID_ARG;
  if (c->pool_kernel > 255) return DKV_ERR_UNSUPPORTED;
  if (c->avg_budget < 1 || c->layer_max < c->avg_budget || c->update_interval < 1) return DKV_ERR_INVALID_ARG;
  if (c->flags & ~DKV_F_ALL) return DKV_ERR_INVALID_ARG;
  if (c->pool_kind != 0 && c->pool_kind != 1) return DKV_ERR_UNSUPPORTED;
  if (c->n_layers > DKV_MAX_LAYERS || c->layer_max > DKV_MAX_LAYER_BUDGET) return DKV_ERR_UNSUPPORTED;
  if (c->head_dim != 64 && c->head_dim != 128) return DKV_ERR_UNSUPPORTED;
  if ((long long)c->window * (c->n_q_heads / c->n_kv_heads) > DKV_MAX_WINDOW_ROWS) return DKV_ERR_UNSUPPORTED;
  if ((long long)c->n_layers * c->batch * c->n_kv_heads * (long long)c->seq_len >= (1ll << 31)) return DKV_ERR_UNSUPPORTED;
  return DKV_OK;
}

// Measurement overrides from the environment, read once per context in dkv_create: an integer inside
// [lo, hi], anything else (unset, not a number, out of range) gives the default.
int env_int(const char* name, int dflt, int lo, int hi) {
  const char* e = getenv(name);
  if (!e || !*e) return dflt;
  char* end = nullptr;
  const long v = strtol(e, &end, 10);
  if (end == e || *end != '\0' || v < lo || v > hi) return dflt;
  return (int)v;
}

int check_layer(const dkv_ctx* c, int layer) {
  if (!c) return DKV_ERR_INVALID_ARG;
  if (layer < 0 || layer >= c->s.L) return DKV_ERR_INVALID_ARG;
  return DKV_OK;
}

// ---- step (1): scores of one layer -------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor [heads][rows][D] seen as (D, rows, heads); boxes of 64 columns x 128 rows, 128-byte swizzle,
// rows past the end of a head read as zero.
bool make_map(CUtensorMap* m, const void* base, int D, int rows, int heads) {
  EncodeTiledFn fn = encode_tiled();
  if (!fn) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)rows, (cuuint64_t)heads};
  const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)rows * D * 2};
  const cuuint32_t box[3] = {64, 128, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

uint32_t make_idesc(int M, int N) {
  // fp32 accumulator, bf16 A and B, both K-major
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Parameters of one sweep over the `nl` consecutive layers that start at `layer` (q, k: their nl device
// pointers); `buf` picks the statistics scratch (jobs in flight rotate).  In sweep 2 every CTA walks its slice of the
// key space from the end to the start: sweep 1 cut the same space into the same slices, so each CTA begins with
// the keys that were streamed last and may still be in L2.
bool make_job(dkv_ctx* c, int mode, int layer, int nl, const void* const* q, const void* const* k, float* scores_out,
              int buf, tc::Maps* maps, tc::Params* p, const float* const* lse = nullptr) {
  const Shape& s = c->s;
  const int heads = s.Bt * s.Hkv;
  memset(maps, 0, sizeof *maps);                           // entries past nl are never read
  for (int i = 0; i < nl; ++i)
    if (!make_map(&maps->q[i], q[i], s.D, s.M, heads) || !make_map(&maps->k[i], k[i], s.D, s.S, heads)) return false;
  if (lse) for (int i = 0; i < nl; ++i) maps->lse[i] = lse[i];
  p->S = s.S; p->P = s.P; p->ws = s.ws; p->M = s.M; p->D = s.D; p->heads = nl * heads; p->half = s.pool / 2;
  p->nl = nl; p->hpl = heads;
  p->back = (mode == tc::kEmit && c->emit_backward) ? 1 : 0;
  p->retain_tiles = (int)((long long)c->retain_mb * (1 << 20) / ((long long)(c->tc_grid > 0 ? c->tc_grid : 1) * tc::kTileKeys * s.D * 2));
  p->wait_cycles = c->wait_cycles;
  p->withhold_tile = c->withhold_sweep == mode ? c->withhold_tile : -1;
  p->tph = (s.S + tc::kTileKeys - 1) / tc::kTileKeys;
  p->nq16 = (s.M + 15) / 16 * 16;
  p->nmblk = (s.M + 127) / 128;
  p->slots = c->tc_slots; p->m_stride = 256;
  p->scale2 = kLog2e / sqrtf((float)s.D);
  p->stats = c->d_tc_stats + (size_t)buf * tc::kMaxGroup * heads * c->tc_slots * 256;
  p->scores = c->d_scores + (size_t)layer * layer_scores(s);
  p->copy_out = scores_out;
  p->status = c->d_status;
  p->stats_grid = c->tc_grid;
  p->mode = mode;
  p->out_scale = (c->cfg.flags & DKV_F_WINDOW_MEAN) ? 1.0f / (float)s.M : 1.0f;
  p->pool_avg = c->cfg.pool_kind == 1;
  p->idesc = mode == tc::kStats ? make_idesc(128, 128) : make_idesc(128, p->nq16);
  return true;
}

// The scoring kernel for two jobs (either may be kNone): the specialised build when every job has exactly 128 window
// rows of 128 dims, the general one otherwise.
void launch_tc(int grid, cudaStream_t st, const tc::Maps& m0, const tc::Maps& m1, const tc::Params& j0, const tc::Params& j1) {
  auto fast = [](const tc::Params& p) { return p.mode == tc::kNone || (p.M == 128 && p.D == 128); };
  if (fast(j0) && fast(j1)) tc::score_tc_kernel<true><<<grid, tc::kThreads, tc::kSmemBytes, st>>>(m0, m1, j0, j1);
  else tc::score_tc_kernel<false><<<grid, tc::kThreads, tc::kSmemBytes, st>>>(m0, m1, j0, j1);
}

// One launch: sweep 2 of the `en` layers from `emit_layer` (if >= 0), then sweep 1 of the `sn` layers from
// `stats_layer` (if >= 0).  In the pass the emit layers are the ones the previous launch streamed.  `sbuf`, `ebuf`: statistics scratch of either job.
int launch_score(dkv_ctx* c, int stats_layer, int sn, const void* const* sq, const void* const* sk, int sbuf,
                 int emit_layer, int en, const void* const* eq, const void* const* ek, int ebuf, float* scores_out,
                 cudaStream_t st, const float* const* emit_lse = nullptr) {
  tc::Maps m0, m1;
  tc::Params j0, j1;
  memset(&j0, 0, sizeof j0); memset(&j1, 0, sizeof j1);
  memset(&m0, 0, sizeof m0); memset(&m1, 0, sizeof m1);
  j0.mode = j1.mode = tc::kNone;
  if (emit_layer >= 0 && !make_job(c, tc::kEmit, emit_layer, en, eq, ek, scores_out, ebuf, &m0, &j0, emit_lse)) return DKV_ERR_CUDA;
  if (stats_layer >= 0 && !make_job(c, tc::kStats, stats_layer, sn, sq, sk, nullptr, sbuf, &m1, &j1)) return DKV_ERR_CUDA;
  ProfScope ps(c, stats_layer >= 0 ? DKV_STEP_SCORE_STATS : DKV_STEP_SCORE_EMIT, 1, st);
  launch_tc(c->tc_grid, st, m0, m1, j0, j1);
  DKV_LAUNCHED(c);
  return DKV_OK;
}

// Sweep 2 alone, with the window rows' normalisers supplied by the caller instead of sweep 1.
int do_score_lse(dkv_ctx* c, int layer, const void* q, const void* k, const float* lse, float* scores_out,
                 cudaStream_t st) {
  tc::Maps maps;
  tc::Params job, none;
  memset(&job, 0, sizeof job); memset(&none, 0, sizeof none);
  none.mode = tc::kNone;
  if (!make_job(c, tc::kEmit, layer, 1, &q, &k, scores_out, layer % 3, &maps, &job, &lse)) return DKV_ERR_CUDA;
  ProfScope ps(c, DKV_STEP_SCORE_EMIT, 1, st);
  launch_tc(c->tc_grid, st, maps, maps, job, none);
  DKV_LAUNCHED(c);
  c->scored[layer] = 1;
  c->selected[layer] = c->gathered[layer] = c->stale[layer] = 0;
  return DKV_OK;
}

int do_score(dkv_ctx* c, int layer, const void* q, const void* k, float* scores_out, cudaStream_t st) {
  int rc = launch_score(c, layer, 1, &q, &k, layer % 3, -1, 0, nullptr, nullptr, 0, nullptr, st);
  if (rc) return rc;
  if ((rc = launch_score(c, -1, 0, nullptr, nullptr, 0, layer, 1, &q, &k, layer % 3, scores_out, st))) return rc;
  c->scored[layer] = 1;
  c->selected[layer] = c->gathered[layer] = c->stale[layer] = 0;
  return DKV_OK;
}

// ---- step (2): per-head top-Bl' ----------------------------------------------------------------
int do_kept_sorted(dkv_ctx* c, int layer, int* sorted_out, cudaStream_t st) {
  const Shape& s = c->s;
  kept_sorted_kernel<<<s.Bt * s.Hkv, kSelThreads, (size_t)((s.P + 31) / 32) * 4, st>>>(
      c->d_idx + (size_t)layer * layer_idx(s), c->d_held, sorted_out, s.P, s.Blc, s.Hkv, s.L, layer);
  DKV_LAUNCHED(c);
  return DKV_OK;
}

int do_select(dkv_ctx* c, int layer, int* sorted_out, int* rank_out, cudaStream_t st) {
  const Shape& s = c->s;
  const size_t heads = (size_t)s.Bt * s.Hkv;
  ProfScope ps(c, DKV_STEP_SELECT, 1, st);
  const float* sc = c->d_scores + (size_t)layer * layer_scores(s);
  int* idx = c->d_idx + (size_t)layer * layer_idx(s);
  unsigned int* lh = c->d_layer_hist + (size_t)layer * s.Bt * kBins;
  DKV_CUDA(c, cudaMemsetAsync(lh, 0, sizeof(unsigned int) * s.Bt * kBins, st));
  if (c->sel_reg)
    select_topk_kernel<true><<<(unsigned)heads, kSelThreads, c->sel_smem, st>>>(
        sc, idx, sorted_out, rank_out, lh, s.P, s.Blc, c->sort_n, c->d_count, s.Hkv, s.L, layer);
  else
    select_topk_kernel<false><<<(unsigned)heads, kSelThreads, c->sel_smem, st>>>(
        sc, idx, sorted_out, rank_out, lh, s.P, s.Blc, c->sort_n, c->d_count, s.Hkv, s.L, layer);
  DKV_LAUNCHED(c);
  c->selected[layer] = 1;
  c->sel_n[layer] = s.Blc;
  c->gathered[layer] = c->stale[layer] = 0;
  return DKV_OK;
}

// ---- step (3): Update_Buffer_Length ------------------------------------------------------------
int do_rebudget(dkv_ctx* c, int l, int* counts_out, cudaStream_t st) {
  const Shape& s = c->s;
  long long k = (long long)s.N * s.Hkv * l;
  const long long pop = (long long)l * s.Hkv * s.P;
  if (k > pop) k = pop;
  ProfScope ps(c, DKV_STEP_REBUDGET, 4, st);
  const size_t per_layer = (size_t)s.Hkv * s.P, cand_stride = (size_t)s.L * per_layer;
  rb_locate_kernel<<<s.Bt, 1024, 0, st>>>(c->d_layer_hist, c->d_rb_state, c->d_rb_above, c->d_rb_hist1,
                                         c->d_rb_above2, c->d_rb_hist2, c->d_cand_n, s.Bt, s.Hkv, s.L, l, s.P, k);
  DKV_LAUNCHED(c);
  int slices = (int)((per_layer + (size_t)kRbThreads * 16 - 1) / ((size_t)kRbThreads * 16));
  if (slices > 64) slices = 64;
  rb_refine1_kernel<<<dim3(slices, l, s.Bt), kRbThreads, 0, st>>>(c->d_scores, c->d_rb_state, c->d_rb_hist1, c->d_cand,
                                                                 c->d_cand_n, s.Bt, per_layer, cand_stride);
  DKV_LAUNCHED(c);
  rb_refine2_kernel<<<dim3(256, s.Bt), kRbThreads, 0, st>>>(c->d_cand, c->d_cand_n, c->d_rb_state, c->d_rb_hist1,
                                                          c->d_rb_above2, c->d_rb_hist2, s.L, cand_stride);
  DKV_LAUNCHED(c);
  const size_t bl = (size_t)s.Bt * s.L;
  rb_budget_kernel<<<s.Bt, 1024, 0, st>>>(c->d_rb_state, c->d_rb_hist1, c->d_rb_above, c->d_rb_above2, c->d_rb_hist2,
                                         c->d_count, c->d_dbg, c->d_dbg + bl, c->d_dbg + 2 * bl, counts_out, s.Bt, s.L, l,
                                         s.Bl, s.N, (c->cfg.flags & DKV_F_PRORATA) != 0, (c->cfg.flags & DKV_F_NORM_MINMAX) != 0);
  DKV_LAUNCHED(c);
  for (int i = 0; i < l; ++i) if (!c->gathered[i]) c->stale[i] = 1;
  return DKV_OK;
}

// ---- step (4): gather / shrink ------------------------------------------------------------------
int do_shrink(dkv_ctx* c, int layer0, int n, void* const* kb, void* const* vb, cudaStream_t st) {
  const Shape& s = c->s;
  LayerPtrs ptrs;
  for (int i = 0; i < n; ++i) { ptrs.kb[layer0 + i] = kb[i]; ptrs.vb[layer0 + i] = vb[i]; }
  ProfScope ps(c, DKV_STEP_SHRINK, 2, st);
  shrink_kernel<<<dim3(s.Bt * s.Hkv, n, 2), kShrinkThreads, 0, st>>>(ptrs, layer0, c->d_count, c->d_held, s.Hkv, s.L, s.ws,
                                                                      s.rows, s.D * 2 / 16);
  DKV_LAUNCHED(c);
  commit_held_kernel<<<(s.Bt * n + 127) / 128, 128, 0, st>>>(c->d_held, c->d_count, s.Bt, s.L, layer0, n);
  DKV_LAUNCHED(c);
  return DKV_OK;
}

int do_gather(dkv_ctx* c, int layer, const void* k_src, const void* v_src, void* kb, void* vb, cudaStream_t st) {
  const Shape& s = c->s;
  const int vec = s.D * 2 / 16, rpb = 256 / vec * kGatherRows;
  const dim3 grid((s.rows + rpb - 1) / rpb, s.Bt * s.Hkv, 2);
  {
  ProfScope ps(c, DKV_STEP_GATHER, 1, st);
  gather_rows_kernel<<<grid, 256, 0, st>>>(static_cast<const uint4*>(k_src), static_cast<const uint4*>(v_src),
                                           static_cast<uint4*>(kb), static_cast<uint4*>(vb),
                                           c->d_idx + (size_t)layer * layer_idx(s), c->sel_n[layer], s.Blc, s.S, s.P, s.ws, s.rows, vec,
                                           c->d_held, s.Hkv, s.L, layer);
  DKV_LAUNCHED(c);
  }
  c->gathered[layer] = 1;
  if (c->stale[layer]) {           // an update ran between select and gather: apply it now
    c->stale[layer] = 0;
    return do_shrink(c, layer, 1, &kb, &vb, st);
  }
  return DKV_OK;
}

int do_reset(dkv_ctx* c, cudaStream_t st) {
  const Shape& s = c->s;
  DKV_CUDA(c, cudaMemsetAsync(c->d_count, 0, sizeof(int) * s.Bt * s.L, st));
  DKV_CUDA(c, cudaMemsetAsync(c->d_held, 0, sizeof(int) * s.Bt * s.L, st));
  DKV_CUDA(c, cudaMemsetAsync(c->d_dbg, 0, sizeof(int) * 3 * s.Bt * s.L, st));
  memset(c->scored, 0, sizeof c->scored);
  memset(c->selected, 0, sizeof c->selected);
  memset(c->gathered, 0, sizeof c->gathered);
  memset(c->stale, 0, sizeof c->stale);
  return DKV_OK;
}

// Algorithm 1's loop.  The scoring launches run back to back on a stream of their own; launch g runs sweep 2
// of layer group g-1 and then sweep 1 of group g (a group = up to `pass_group` consecutive layers, so that the
// fixed cost of a launch and of a job is paid once per group).  Everything that consumes a layer's scores (select,
// gather, and every m layers rebudget + shrink) runs on side streams behind events, layers alternating between
// two of them, so that it overlaps the scoring of the following groups.  `st` rejoins all of them at the end.
// With `lse` (the window rows' log-denominators of every layer) sweep 1 is not needed: launch g runs sweep 2 of group g.
int do_pass(dkv_ctx* c, const void* const* q, const void* const* k, const void* const* v, const float* const* lse,
            void* const* kb, void* const* vb, cudaStream_t st) {
  const Shape& s = c->s;
  int rc = do_reset(c, st);
  if (rc) return rc;
  DKV_CUDA(c, cudaEventRecord(c->ev_fork, st));
  for (int i = 0; i < c->n_side; ++i) DKV_CUDA(c, cudaStreamWaitEvent(c->side[i], c->ev_fork, 0));
  DKV_CUDA(c, cudaStreamWaitEvent(c->hi, c->ev_fork, 0));
  DKV_CUDA(c, cudaStreamWaitEvent(c->upd, c->ev_fork, 0));
  cudaStream_t caller = st;
  st = c->hi;
  // Group sizes: `pass_group` layers each.  (With DKV_PASS_TAPER=1 they halve towards the end, so that less work
  // is left for after the last launch; with four select streams that tail is as short either way.)
  int first[DKV_MAX_LAYERS + 2], groups = 0;
  for (int done = 0; done < s.L;) {
    int n = c->pass_taper ? (s.L - done) / 2 : c->pass_group;
    if (n > c->pass_group) n = c->pass_group;
    if (n > s.L - done) n = s.L - done;
    if (n < 1) n = 1;
    first[groups++] = done;
    done += n;
  }
  first[groups] = s.L;
  for (int g = lse ? 1 : 0; g <= groups; ++g) {
    const int sl = g < groups && !lse ? first[g] : -1, sn = sl >= 0 ? first[g + 1] - first[g] : 0;
    const int e0 = g > 0 ? first[g - 1] : -1, en = g > 0 ? first[g] - first[g - 1] : 0;
    if ((rc = launch_score(c, sl, sn, sl >= 0 ? q + sl : nullptr, sl >= 0 ? k + sl : nullptr, g % 3, e0, en,
                           e0 >= 0 ? q + e0 : nullptr, e0 >= 0 ? k + e0 : nullptr, (g + 2) % 3, nullptr, st,
                           lse && e0 >= 0 ? lse + e0 : nullptr)))
      return rc;
    if (e0 < 0) continue;
    DKV_CUDA(c, cudaEventRecord(c->ev_scored[e0], st));
    for (int el = e0; el < e0 + en; ++el) {
      c->scored[el] = 1;
      cudaStream_t sd = c->side[el % c->n_side];
      DKV_CUDA(c, cudaStreamWaitEvent(sd, c->ev_scored[e0], 0));
      if ((rc = do_select(c, el, nullptr, nullptr, sd))) return rc;
      DKV_CUDA(c, cudaEventRecord(c->ev_picked[el], sd));
      if ((rc = do_gather(c, el, k[el], v[el], kb[el], vb[el], sd))) return rc;
      DKV_CUDA(c, cudaEventRecord(c->ev_selected[el], sd));
      const bool update = ((el + 1) % s.m == 0) || (el + 1 == s.L && s.L % s.m != 0);
      if (update) {
        // The rebudget needs every earlier layer selected (every select stream, each in layer order), the shrink
        // also gathered; the previous update precedes it on the same stream.  Later layers' select and gather
        // do not wait for it: an update changes the counts and buffers of the layers before it only.
        for (int b = 0; b < c->n_side && b <= el; ++b) DKV_CUDA(c, cudaStreamWaitEvent(c->upd, c->ev_picked[el - b], 0));
        if ((rc = do_rebudget(c, el + 1, nullptr, c->upd))) return rc;
        for (int b = 0; b < c->n_side && b <= el; ++b) DKV_CUDA(c, cudaStreamWaitEvent(c->upd, c->ev_selected[el - b], 0));
        if ((rc = do_shrink(c, 0, el + 1, kb, vb, c->upd))) return rc;
      }
    }
  }
  for (int i = 0; i < c->n_side; ++i) {
    DKV_CUDA(c, cudaEventRecord(c->ev_join[i], c->side[i]));
    DKV_CUDA(c, cudaStreamWaitEvent(caller, c->ev_join[i], 0));
  }
  DKV_CUDA(c, cudaEventRecord(c->ev_join[kSideStreams], c->hi));
  DKV_CUDA(c, cudaStreamWaitEvent(caller, c->ev_join[kSideStreams], 0));
  DKV_CUDA(c, cudaEventRecord(c->ev_update, c->upd));
  DKV_CUDA(c, cudaStreamWaitEvent(caller, c->ev_update, 0));
  return DKV_OK;
}

void free_all(dkv_ctx* c) {
  cudaFree(c->d_scores); cudaFree(c->d_idx); cudaFree(c->d_count);
  cudaFree(c->d_held); cudaFree(c->d_dbg); cudaFree(c->d_rb_state); cudaFree(c->d_rb_above); cudaFree(c->d_rb_hist1);
  cudaFree(c->d_rb_above2); cudaFree(c->d_rb_hist2); cudaFree(c->d_layer_hist);
  cudaFree(c->d_cand); cudaFree(c->d_cand_n); cudaFree(c->d_status); cudaFree(c->d_tc_stats);
  cudaFree(c->d_dec_scratch); cudaFree(c->d_dec_tickets);
  for (int i = 0; i < kSideStreams; ++i) if (c->side[i]) cudaStreamDestroy(c->side[i]);
  if (c->hi) cudaStreamDestroy(c->hi);
  if (c->pass_exec) cudaGraphExecDestroy(c->pass_exec);
  delete c->pass_key;
  if (c->gstream) cudaStreamDestroy(c->gstream);
  if (c->ev_gfork) cudaEventDestroy(c->ev_gfork);
  if (c->ev_gjoin) cudaEventDestroy(c->ev_gjoin);
  if (c->upd) cudaStreamDestroy(c->upd);
  for (int i = 0; i <= kSideStreams; ++i) if (c->ev_join[i]) cudaEventDestroy(c->ev_join[i]);
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  if (c->ev_update) cudaEventDestroy(c->ev_update);
  for (int l = 0; l < DKV_MAX_LAYERS; ++l) {
    if (c->ev_scored[l]) cudaEventDestroy(c->ev_scored[l]);
    if (c->ev_selected[l]) cudaEventDestroy(c->ev_selected[l]);
    if (c->ev_picked[l]) cudaEventDestroy(c->ev_picked[l]);
  }
  if (c->prof_recs) {
    for (ProfRec& r : *c->prof_recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    delete c->prof_recs;
  }
  if (c->staged) {
    for (int i = 0; i < 2; ++i) {
      cudaFree(c->st_q[i]); cudaFree(c->st_k[i]); cudaFree(c->st_v[i]);
      cudaEventDestroy(c->ev_copied[i]); cudaEventDestroy(c->ev_consumed[i]);
    }
    for (int l = 0; l < c->s.L; ++l) { cudaFree(c->st_kb[l]); cudaFree(c->st_vb[l]); }
    cudaStreamDestroy(c->st_copy); cudaStreamDestroy(c->st_comp);
  }
}

int ensure_staging(dkv_ctx* c) {
  if (c->staged) return DKV_OK;
  const Shape& s = c->s;
  for (int i = 0; i < 2; ++i) {
    DKV_CUDA(c, cudaMalloc(&c->st_q[i], layer_q_bytes(s)));
    DKV_CUDA(c, cudaMalloc(&c->st_k[i], layer_kv_bytes(s)));
    DKV_CUDA(c, cudaMalloc(&c->st_v[i], layer_kv_bytes(s)));
    DKV_CUDA(c, cudaEventCreateWithFlags(&c->ev_copied[i], cudaEventDisableTiming));
    DKV_CUDA(c, cudaEventCreateWithFlags(&c->ev_consumed[i], cudaEventDisableTiming));
  }
  for (int l = 0; l < s.L; ++l) {
    DKV_CUDA(c, cudaMalloc(&c->st_kb[l], layer_buf_bytes(s)));
    DKV_CUDA(c, cudaMalloc(&c->st_vb[l], layer_buf_bytes(s)));
  }
  DKV_CUDA(c, cudaStreamCreateWithFlags(&c->st_copy, cudaStreamNonBlocking));
  DKV_CUDA(c, cudaStreamCreateWithFlags(&c->st_comp, cudaStreamNonBlocking));
  c->staged = true;
  return DKV_OK;
}

}  // namespace

extern "C" {

int dkv_version(void) { return 1000; }

const char* dkv_strerror(int code) {
  switch (code) {
    case DKV_OK: return "ok";
    case DKV_ERR_INVALID_ARG: return "invalid argument";
    case DKV_ERR_STATE: return "call out of order for this layer";
    case DKV_ERR_CUDA: return "CUDA runtime error";
    case DKV_ERR_TIMEOUT: return "device-side wait timed out";
    case DKV_ERR_UNSUPPORTED: return "shape not supported";
    case DKV_ERR_NOMEM: return "out of memory";
    case DKV_ERR_TOO_LARGE: return "problem needs more scratch than the static array holds";
    default: return "unknown error";
  }
}

int dkv_create(const dkv_config* cfg, dkv_ctx** out) {
  if (!out) return DKV_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = validate(cfg);
  if (rc) return rc;
  dkv_ctx* c = new (std::nothrow) dkv_ctx;
  if (!c) return DKV_ERR_NOMEM;
  memset(c, 0, sizeof *c);
  c->cfg = *cfg;
  c->prof_recs = new (std::nothrow) std::vector<ProfRec>();
  if (!c->prof_recs) { delete c; return DKV_ERR_NOMEM; }
  Shape& s = c->s;
  s.L = cfg->n_layers; s.Hq = cfg->n_q_heads; s.Hkv = cfg->n_kv_heads; s.D = cfg->head_dim; s.Bt = cfg->batch;
  s.S = cfg->seq_len; s.ws = cfg->window; s.pool = cfg->pool_kernel; s.N = cfg->avg_budget; s.Bl = cfg->layer_max;
  s.m = cfg->update_interval;
  s.G = s.Hq / s.Hkv; s.P = s.S - s.ws; s.M = s.ws * s.G; s.Blc = s.Bl < s.P ? s.Bl : s.P; s.rows = s.Blc + s.ws;
  const int heads = s.Bt * s.Hkv;
  c->sort_n = 2;
  while (c->sort_n < s.Blc) c->sort_n <<= 1;

  cudaError_t e = cudaGetDevice(&c->device);
  {
    int sms = 0;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
    c->n_sms = sms > 0 ? sms : 1;
    const int tph = (s.S + tc::kTileKeys - 1) / tc::kTileKeys;
    const long long total_tiles = (long long)heads * tph;
    // leave some SMs to the select / gather / update kernels that dkv_run_prefill_pass runs beside the scoring:
    // with grouped launches up to four layers' selects (one CTA per head) are in flight at once
    int side = 4 * heads < c->n_sms * 2 / 9 ? 4 * heads : c->n_sms * 2 / 9;
    side = env_int("DKV_SIDE_SMS", side, 0, c->n_sms - 1);
    int score_sms = c->n_sms - side;
    if (score_sms < 1) score_sms = 1;
    c->tc_grid = (int)(total_tiles < score_sms ? total_tiles : score_sms);
    int slots = 1;
    for (int nl = 1; nl <= tc::kMaxGroup; ++nl)           // a job may cover up to kMaxGroup layers (the pass groups them)
      for (int bh = 0; bh < nl * heads; ++bh) {
        const int lo = tc::tile_owner((long long)bh * tph, nl * total_tiles, c->tc_grid);
        const int hi = tc::tile_owner((long long)(bh + 1) * tph - 1, nl * total_tiles, c->tc_grid);
        if (hi - lo + 1 > slots) slots = hi - lo + 1;
      }
    c->tc_slots = slots;
    // layers per scoring launch of the pass: enough that a CTA's share of a job is some tens of tiles
    c->pass_group = env_int("DKV_PASS_GROUP", total_tiles / c->tc_grid < 8 ? tc::kMaxGroup : 4, 1, tc::kMaxGroup);
    c->pass_taper = env_int("DKV_PASS_TAPER", 0, 0, 1);
    c->n_side = env_int("DKV_SIDE_STREAMS", kSideStreams, 1, kSideStreams);
    c->emit_backward = env_int("DKV_EMIT_FORWARD", 0, 0, 1) == 0;
    // Sweep 2 starts on the keys sweep 1 streamed last: that much of a job (4/7 of L2, 72 of 126 MB) is loaded with
    // an evict-last policy, every other key tile and the gather's rows evict-first, so that neither the rest of the
    // stream nor the side kernels' traffic pushes it out before it is read again.
    int l2_bytes = 0;
    if (cudaDeviceGetAttribute(&l2_bytes, cudaDevAttrL2CacheSize, c->device) != cudaSuccess) l2_bytes = 0;
    c->retain_mb = c->emit_backward ? env_int("DKV_L2_RETAIN_MB", (int)(((long long)l2_bytes * 4 / 7) >> 20), 0, 1024) : 0;
    c->host_v_staged = env_int("DKV_HOST_V_STAGED", 0, 0, 1) != 0;
    c->host_h2d = c->host_d2h = 0;
    c->wait_cycles = tc::kDefaultWaitCycles;
    c->withhold_sweep = c->withhold_tile = -1;
  }
  const size_t bl = (size_t)s.Bt * s.L;
#define TRY(call) if (e == cudaSuccess) e = (call)
  TRY(cudaMalloc(&c->d_scores, sizeof(float) * s.L * layer_scores(s)));
  TRY(cudaMalloc(&c->d_idx, sizeof(int) * s.L * layer_idx(s)));
  TRY(cudaMalloc(&c->d_count, sizeof(int) * bl));
  TRY(cudaMalloc(&c->d_held, sizeof(int) * bl));
  TRY(cudaMalloc(&c->d_dbg, sizeof(int) * 3 * bl));
  TRY(cudaMalloc(&c->d_rb_state, sizeof(RbState) * s.Bt));
  TRY(cudaMalloc(&c->d_rb_above, sizeof(unsigned int) * bl));
  TRY(cudaMalloc(&c->d_rb_above2, sizeof(unsigned int) * bl));
  TRY(cudaMalloc(&c->d_rb_hist1, sizeof(unsigned int) * s.Bt * kBins));
  TRY(cudaMalloc(&c->d_rb_hist2, sizeof(unsigned int) * bl * 1024));
  TRY(cudaMalloc(&c->d_layer_hist, sizeof(unsigned int) * s.L * s.Bt * kBins));
  TRY(cudaMalloc(&c->d_cand, sizeof(uint2) * s.L * layer_scores(s)));
  TRY(cudaMalloc(&c->d_cand_n, sizeof(unsigned int) * s.Bt));
  TRY(cudaMalloc(&c->d_tc_stats, sizeof(float2) * 3 * tc::kMaxGroup * heads * c->tc_slots * 256));
  TRY(cudaFuncSetAttribute(tc::score_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes));
  TRY(cudaFuncSetAttribute(tc::score_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes));
  for (int i = 0; i < kSideStreams; ++i) TRY(cudaStreamCreateWithFlags(&c->side[i], cudaStreamNonBlocking));
  TRY(cudaStreamCreateWithFlags(&c->gstream, cudaStreamNonBlocking));
  TRY(cudaEventCreateWithFlags(&c->ev_gfork, cudaEventDisableTiming));
  TRY(cudaEventCreateWithFlags(&c->ev_gjoin, cudaEventDisableTiming));
  c->pass_key = new (std::nothrow) std::vector<const void*>();
  if (!c->pass_key) { free_all(c); delete c; return DKV_ERR_NOMEM; }
  c->use_graph = env_int("DKV_NO_GRAPH", 0, 0, 1) == 0;
  TRY(cudaStreamCreateWithFlags(&c->upd, cudaStreamNonBlocking));
  {
    int least = 0, greatest = 0;
    TRY(cudaDeviceGetStreamPriorityRange(&least, &greatest));
    TRY(cudaStreamCreateWithPriority(&c->hi, cudaStreamNonBlocking, greatest));
  }
  for (int i = 0; i <= kSideStreams; ++i) TRY(cudaEventCreateWithFlags(&c->ev_join[i], cudaEventDisableTiming));
  TRY(cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming));
  TRY(cudaEventCreateWithFlags(&c->ev_update, cudaEventDisableTiming));
  for (int l = 0; l < s.L; ++l) {
    TRY(cudaEventCreateWithFlags(&c->ev_scored[l], cudaEventDisableTiming));
    TRY(cudaEventCreateWithFlags(&c->ev_selected[l], cudaEventDisableTiming));
    TRY(cudaEventCreateWithFlags(&c->ev_picked[l], cudaEventDisableTiming));
  }
  TRY(cudaMalloc(&c->d_status, sizeof(int) * 8));
  TRY(cudaMemset(c->d_status, 0, sizeof(int) * 8));
  TRY(cudaMemset(c->d_count, 0, sizeof(int) * bl));
  TRY(cudaMemset(c->d_held, 0, sizeof(int) * bl));
  TRY(cudaMemset(c->d_dbg, 0, sizeof(int) * 3 * bl));
  {
    c->sel_reg = (s.P + kSelThreads - 1) / kSelThreads <= kRegChunk;
    c->sel_smem = (size_t)c->sort_n * 8 + (size_t)s.Blc * 4;
  }
  // The attribute belongs to the function, not to this context: always the most any valid configuration needs
  // (sort keys 8 B and positions 4 B for DKV_MAX_LAYER_BUDGET entries), so that contexts do not undo each other.
  TRY(cudaFuncSetAttribute(select_topk_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSelMaxSmem));
  TRY(cudaFuncSetAttribute(select_topk_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSelMaxSmem));
#undef TRY
  if (e != cudaSuccess) {
    rc = e == cudaErrorMemoryAllocation ? DKV_ERR_NOMEM : DKV_ERR_CUDA;
    cudaGetLastError();
    free_all(c);
    delete c;
    return rc;
  }
  *out = c;
  return DKV_OK;
}

int dkv_destroy(dkv_ctx* c) {
  if (!c) return DKV_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  free_all(c);
  delete c;
  return DKV_OK;
}

int dkv_reset(dkv_ctx* c, void* stream) {
  if (!c) return DKV_ERR_INVALID_ARG;
  return do_reset(c, as_stream(stream));
}

int dkv_score(dkv_ctx* c, int32_t layer, const void* q_win, const void* k, float* scores_out, void* stream) {
  int rc = check_layer(c, layer);
  if (rc) return rc;
  if (!q_win || !k || !aligned16(q_win) || !aligned16(k) || !aligned16(scores_out)) return DKV_ERR_INVALID_ARG;
  return do_score(c, layer, q_win, k, scores_out, as_stream(stream));
}

int dkv_score_lse(dkv_ctx* c, int32_t layer, const void* q_win, const void* k, const float* lse, float* scores_out,
                  void* stream) {
  int rc = check_layer(c, layer);
  if (rc) return rc;
  if (!q_win || !k || !lse || !aligned16(q_win) || !aligned16(k) || !aligned16(scores_out) || ((uintptr_t)lse & 3))
    return DKV_ERR_INVALID_ARG;
  return do_score_lse(c, layer, q_win, k, lse, scores_out, as_stream(stream));
}

int dkv_set_scores(dkv_ctx* c, int32_t layer, const float* scores, void* stream) {
  int rc = check_layer(c, layer);
  if (rc) return rc;
  if (!scores) return DKV_ERR_INVALID_ARG;
  const size_t n = layer_scores(c->s);
  DKV_CUDA(c, cudaMemcpyAsync(c->d_scores + (size_t)layer * n, scores, n * sizeof(float), cudaMemcpyDeviceToDevice,
                              as_stream(stream)));
  c->scored[layer] = 1;
  c->selected[layer] = c->gathered[layer] = c->stale[layer] = 0;
  return DKV_OK;
}

int dkv_select_topk(dkv_ctx* c, int32_t layer, int32_t* idx_out, int32_t* rank_out, void* stream) {
  int rc = check_layer(c, layer);
  if (rc) return rc;
  if (!c->scored[layer]) return DKV_ERR_STATE;
  return do_select(c, layer, idx_out, rank_out, as_stream(stream));
}

int dkv_rebudget(dkv_ctx* c, int32_t upto_layer, int32_t* counts_out, void* stream) {
  if (!c || upto_layer < 1 || upto_layer > c->s.L) return DKV_ERR_INVALID_ARG;
  for (int i = 0; i < upto_layer; ++i) if (!c->scored[i] || c->selected[i] != 1) return DKV_ERR_STATE;
  return do_rebudget(c, upto_layer, counts_out, as_stream(stream));
}

int dkv_compact(dkv_ctx* c, int32_t layer, const void* k_src, const void* v_src, void* kb, void* vb, int32_t* len_out,
                void* stream) {
  int rc = check_layer(c, layer);
  if (rc) return rc;
  if (!kb || !vb || !aligned16(kb) || !aligned16(vb)) return DKV_ERR_INVALID_ARG;
  if ((k_src == nullptr) != (v_src == nullptr)) return DKV_ERR_INVALID_ARG;
  if (!aligned16(k_src) || !aligned16(v_src)) return DKV_ERR_INVALID_ARG;
  cudaStream_t st = as_stream(stream);
  if (k_src) {
    if (!c->selected[layer]) return DKV_ERR_STATE;
    rc = do_gather(c, layer, k_src, v_src, kb, vb, st);
  } else {
    if (!c->gathered[layer]) return DKV_ERR_STATE;
    rc = do_shrink(c, layer, 1, &kb, &vb, st);
  }
  if (rc) return rc;
  if (len_out) {
    const Shape& s = c->s;
    write_len_kernel<<<(s.Bt * s.Hkv + 127) / 128, 128, 0, st>>>(len_out, c->d_held, s.Bt, s.Hkv, s.L, layer, s.ws);
    DKV_LAUNCHED(c);
  }
  return DKV_OK;
}

int dkv_compact_all(dkv_ctx* c, int32_t upto_layer, void* const* kb, void* const* vb, void* stream) {
  if (!c || !kb || !vb || upto_layer < 1 || upto_layer > c->s.L) return DKV_ERR_INVALID_ARG;
  for (int i = 0; i < upto_layer; ++i) {
    if (!kb[i] || !vb[i] || !aligned16(kb[i]) || !aligned16(vb[i])) return DKV_ERR_INVALID_ARG;
    if (!c->gathered[i]) return DKV_ERR_STATE;
  }
  return do_shrink(c, 0, upto_layer, kb, vb, as_stream(stream));
}

static int run_pass(dkv_ctx* c, const void* const* q_win, const void* const* k, const void* const* v,
                    const float* const* lse, void* const* kb, void* const* vb, void* stream) {
  if (!c || !q_win || !k || !v || !kb || !vb) return DKV_ERR_INVALID_ARG;
  for (int l = 0; l < c->s.L; ++l) {
    if (!q_win[l] || !k[l] || !v[l] || !kb[l] || !vb[l]) return DKV_ERR_INVALID_ARG;
    if (!aligned16(q_win[l]) || !aligned16(k[l]) || !aligned16(v[l]) || !aligned16(kb[l]) || !aligned16(vb[l]))
      return DKV_ERR_INVALID_ARG;
    if (lse && (!lse[l] || ((uintptr_t)lse[l] & 3))) return DKV_ERR_INVALID_ARG;
  }
  cudaStream_t st = as_stream(stream);
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) { cudaGetLastError(); cap = cudaStreamCaptureStatusNone; }
  // per-step profiling needs its events between the launches; a caller that is capturing gets the plain calls
  if (!c->use_graph || c->prof_on || cap != cudaStreamCaptureStatusNone) return do_pass(c, q_win, k, v, lse, kb, vb, st);

  std::vector<const void*> key;
  key.reserve(6 * (size_t)c->s.L);
  for (int l = 0; l < c->s.L; ++l) {
    key.push_back(q_win[l]); key.push_back(k[l]); key.push_back(v[l]); key.push_back(kb[l]); key.push_back(vb[l]);
    key.push_back(lse ? lse[l] : nullptr);
  }
  if (!c->pass_exec || *c->pass_key != key) {
    // first call with these buffers: record the whole pass (all streams of do_pass fork from and rejoin gstream)
    if (c->pass_exec) { cudaGraphExecDestroy(c->pass_exec); c->pass_exec = nullptr; }
    const long long before = c->launches;
    cudaGraph_t graph = nullptr;
    DKV_CUDA(c, cudaStreamBeginCapture(c->gstream, cudaStreamCaptureModeThreadLocal));
    const int rc = do_pass(c, q_win, k, v, lse, kb, vb, c->gstream);
    const cudaError_t e = cudaStreamEndCapture(c->gstream, &graph);
    if (rc != DKV_OK || e != cudaSuccess || !graph) {
      if (graph) cudaGraphDestroy(graph);
      cudaGetLastError();
      c->launches = before;
      c->use_graph = false;                         // not capturable here: run the plain calls from now on
      return do_pass(c, q_win, k, v, lse, kb, vb, st);
    }
    c->pass_launches = c->launches - before;
    c->launches = before;
    const cudaError_t ei = cudaGraphInstantiate(&c->pass_exec, graph, 0);
    cudaGraphDestroy(graph);
    if (ei != cudaSuccess) {
      cudaGetLastError();
      c->pass_exec = nullptr; c->use_graph = false;
      return do_pass(c, q_win, k, v, lse, kb, vb, st);
    }
    *c->pass_key = key;
  }
  DKV_CUDA(c, cudaEventRecord(c->ev_gfork, st));
  DKV_CUDA(c, cudaStreamWaitEvent(c->gstream, c->ev_gfork, 0));
  DKV_CUDA(c, cudaGraphLaunch(c->pass_exec, c->gstream));
  DKV_CUDA(c, cudaEventRecord(c->ev_gjoin, c->gstream));
  DKV_CUDA(c, cudaStreamWaitEvent(st, c->ev_gjoin, 0));
  c->launches += c->pass_launches;
  for (int l = 0; l < c->s.L; ++l) { c->scored[l] = c->selected[l] = c->gathered[l] = 1; c->stale[l] = 0; c->sel_n[l] = c->s.Blc; }
  return DKV_OK;
}

int dkv_run_prefill_pass(dkv_ctx* c, const void* const* q_win, const void* const* k, const void* const* v,
                         void* const* kb, void* const* vb, void* stream) {
  return run_pass(c, q_win, k, v, nullptr, kb, vb, stream);
}

int dkv_run_prefill_pass_lse(dkv_ctx* c, const void* const* q_win, const void* const* k, const void* const* v,
                             const float* const* lse, void* const* kb, void* const* vb, void* stream) {
  if (!lse) return DKV_ERR_INVALID_ARG;
  return run_pass(c, q_win, k, v, lse, kb, vb, stream);
}

int dkv_run_prefill_pass_host(dkv_ctx* c, const void* const* q_win, const void* const* k, const void* const* v,
                              void* const* kb, void* const* vb, int32_t* counts_out) {
  if (!c || !q_win || !k || !v || !kb || !vb) return DKV_ERR_INVALID_ARG;
  const Shape& s = c->s;
  for (int l = 0; l < s.L; ++l)
    if (!q_win[l] || !k[l] || !v[l] || !kb[l] || !vb[l]) return DKV_ERR_INVALID_ARG;
  int rc = ensure_staging(c);
  if (rc) return rc;
  cudaStream_t cp = c->st_copy, st = c->st_comp;
  if ((rc = do_reset(c, st))) return rc;
  // Only the kept rows of V are ever needed on the device (count + ws of S per head).  Where the caller's V is
  // page-locked host memory that kernels can address, the gather reads exactly those rows over the bus instead of
  // V being copied in full first; pageable memory (or DKV_HOST_V_STAGED=1) takes the full copy.
  const void* v_dev[DKV_MAX_LAYERS];
  for (int l = 0; l < s.L; ++l) {
    v_dev[l] = nullptr;
    if (c->host_v_staged) continue;
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, v[l]) == cudaSuccess && at.type == cudaMemoryTypeHost && at.devicePointer && aligned16(at.devicePointer))
      v_dev[l] = at.devicePointer;
    else
      cudaGetLastError();                      // an unregistered pointer is not an error here
  }
  const long long row_bytes = (long long)s.D * 2;
  long long h2d = 0;
  for (int l = 0; l < s.L; ++l) {
    const int slot = l & 1;
    if (l >= 2) DKV_CUDA(c, cudaStreamWaitEvent(cp, c->ev_consumed[slot], 0));
    DKV_CUDA(c, cudaMemcpyAsync(c->st_q[slot], q_win[l], layer_q_bytes(s), cudaMemcpyHostToDevice, cp));
    DKV_CUDA(c, cudaMemcpyAsync(c->st_k[slot], k[l], layer_kv_bytes(s), cudaMemcpyHostToDevice, cp));
    h2d += (long long)layer_q_bytes(s) + (long long)layer_kv_bytes(s);
    if (!v_dev[l]) {
      DKV_CUDA(c, cudaMemcpyAsync(c->st_v[slot], v[l], layer_kv_bytes(s), cudaMemcpyHostToDevice, cp));
      h2d += (long long)layer_kv_bytes(s);
    }
    DKV_CUDA(c, cudaEventRecord(c->ev_copied[slot], cp));
    DKV_CUDA(c, cudaStreamWaitEvent(st, c->ev_copied[slot], 0));
    if ((rc = do_score(c, l, c->st_q[slot], c->st_k[slot], nullptr, st))) return rc;
    if ((rc = do_select(c, l, nullptr, nullptr, st))) return rc;
    if ((rc = do_gather(c, l, c->st_k[slot], v_dev[l] ? v_dev[l] : c->st_v[slot], c->st_kb[l], c->st_vb[l], st))) return rc;
    if (v_dev[l]) h2d += (long long)(c->sel_n[l] + s.ws) * s.Bt * s.Hkv * row_bytes;
    DKV_CUDA(c, cudaEventRecord(c->ev_consumed[slot], st));
    const bool update = ((l + 1) % s.m == 0) || (l + 1 == s.L && s.L % s.m != 0);
    if (update) {
      if ((rc = do_rebudget(c, l + 1, nullptr, st))) return rc;
      if ((rc = do_shrink(c, 0, l + 1, c->st_kb, c->st_vb, st))) return rc;
    }
  }
  // The final counts come back first; then only the valid rows of every head (count + ws of the fixed stride)
  // are copied out, one strided copy per (layer, sample, tensor).
  std::vector<int> counts((size_t)s.Bt * s.L);
  DKV_CUDA(c, cudaMemcpyAsync(counts.data(), c->d_count, sizeof(int) * s.Bt * s.L, cudaMemcpyDeviceToHost, st));
  DKV_CUDA(c, cudaStreamSynchronize(st));
  const size_t row = (size_t)s.D * 2, head_pitch = (size_t)s.rows * row, sample = (size_t)s.Hkv * head_pitch;
  for (int l = 0; l < s.L; ++l)
    for (int b = 0; b < s.Bt; ++b) {
      const size_t valid = (size_t)(counts[(size_t)b * s.L + l] + s.ws) * row;
      DKV_CUDA(c, cudaMemcpy2DAsync(static_cast<char*>(kb[l]) + b * sample, head_pitch,
                                    static_cast<const char*>(c->st_kb[l]) + b * sample, head_pitch, valid, s.Hkv,
                                    cudaMemcpyDeviceToHost, st));
      DKV_CUDA(c, cudaMemcpy2DAsync(static_cast<char*>(vb[l]) + b * sample, head_pitch,
                                    static_cast<const char*>(c->st_vb[l]) + b * sample, head_pitch, valid, s.Hkv,
                                    cudaMemcpyDeviceToHost, st));
    }
  if (counts_out) memcpy(counts_out, counts.data(), sizeof(int) * s.Bt * s.L);
  long long d2h = (long long)sizeof(int) * s.Bt * s.L;
  for (size_t i = 0; i < counts.size(); ++i) d2h += 2ll * (counts[i] + s.ws) * s.Hkv * row_bytes;
  c->host_h2d = h2d; c->host_d2h = d2h;
  DKV_CUDA(c, cudaStreamSynchronize(cp));
  DKV_CUDA(c, cudaStreamSynchronize(st));
  return DKV_OK;
}

int dkv_host_pass_bytes(dkv_ctx* c, int64_t* h2d, int64_t* d2h) {
  if (!c || !h2d || !d2h) return DKV_ERR_INVALID_ARG;
  *h2d = c->host_h2d; *d2h = c->host_d2h;
  return DKV_OK;
}

int dkv_apply_policy(dkv_ctx* c, int32_t policy, int32_t* counts_out, void* stream) {
  if (!c || (policy != DKV_POLICY_UNIFORM && policy != DKV_POLICY_PYRAMID)) return DKV_ERR_INVALID_ARG;
  const Shape& s = c->s;
  for (int i = 0; i < s.L; ++i) if (!c->selected[i]) return DKV_ERR_STATE;
  policy_counts_kernel<<<(s.Bt * s.L + 127) / 128, 128, 0, as_stream(stream)>>>(c->d_count, counts_out, s.Bt, s.L, s.N, policy);
  DKV_LAUNCHED(c);
  for (int i = 0; i < s.L; ++i) if (!c->gathered[i]) c->stale[i] = 1;
  return DKV_OK;
}

int dkv_select_positions(dkv_ctx* c, int32_t layer, int32_t n_sink, int32_t n_recent, void* stream) {
  int rc = check_layer(c, layer);
  if (rc) return rc;
  const Shape& s = c->s;
  if (n_sink < 0 || n_recent < 0) return DKV_ERR_INVALID_ARG;
  if (n_sink > s.P) n_sink = s.P;
  if (n_recent > s.P) n_recent = s.P;
  const int first_recent = s.P - n_recent > n_sink ? s.P - n_recent : n_sink;
  const int n = n_sink + (s.P - first_recent);
  if (n > s.Blc) return DKV_ERR_INVALID_ARG;
  {
    const dim3 grid((n + 255) / 256 > 0 ? (n + 255) / 256 : 1, s.Bt * s.Hkv);
    positions_kernel<<<grid, 256, 0, as_stream(stream)>>>(c->d_idx + (size_t)layer * layer_idx(s), c->d_count, s.P, s.Blc, n_sink,
                                                         first_recent, n, s.Hkv, s.L, layer);
    DKV_LAUNCHED(c);
  }
  c->selected[layer] = 2;
  c->sel_n[layer] = n;
  c->gathered[layer] = c->stale[layer] = 0;
  return DKV_OK;
}

int dkv_decode_attend(dkv_ctx* c, int32_t layer0, int32_t n_layers, int32_t nq, const void* const* q_dec,
                      const void* const* kb, const void* const* vb, float* const* out, void* stream) {
  if (!c || !q_dec || !kb || !vb || !out) return DKV_ERR_INVALID_ARG;
  const Shape& s = c->s;
  if (layer0 < 0 || n_layers < 1 || layer0 + n_layers > s.L || nq < 1 || (long long)nq * s.G > 64) return DKV_ERR_INVALID_ARG;
  for (int i = 0; i < n_layers; ++i) {
    if (!q_dec[i] || !kb[i] || !vb[i] || !out[i]) return DKV_ERR_INVALID_ARG;
    if (!aligned16(q_dec[i]) || !aligned16(kb[i]) || !aligned16(vb[i]) || !aligned16(out[i])) return DKV_ERR_INVALID_ARG;
    if (!c->gathered[layer0 + i]) return DKV_ERR_STATE;
  }
  cudaStream_t st = as_stream(stream);
  const int BH = s.Bt * s.Hkv, GQ = s.G * nq;
  if (!c->d_dec_tickets) {
    DKV_CUDA(c, cudaMalloc(&c->d_dec_tickets, sizeof(unsigned int) * s.L * BH));
    DKV_CUDA(c, cudaMemset(c->d_dec_tickets, 0, sizeof(unsigned int) * s.L * BH));
  }
  for (int l0 = 0; l0 < n_layers; l0 += kDecMaxLayers) {
    const int nl = n_layers - l0 < kDecMaxLayers ? n_layers - l0 : kDecMaxLayers;
    // a launch over few heads is latency-bound: one resident wave of thread blocks (two fit an SM); one over many
    // heads is bandwidth-bound: a few waves, for more loads in flight; every block gets at least a few dozen rows
    const int waves = BH * nl >= c->n_sms ? 4 : 2;
    int splits = (waves * c->n_sms + BH * nl - 1) / (BH * nl);
    const int most = (s.rows + 31) / 32;
    if (splits > most) splits = most;
    if (splits > 64) splits = 64;
    if (splits < 1) splits = 1;
    const size_t need = (size_t)nl * BH * splits * GQ * (s.D + 2);
    if (need > c->dec_scratch_floats) {
      if (c->d_dec_scratch) { DKV_CUDA(c, cudaDeviceSynchronize()); cudaFree(c->d_dec_scratch); c->d_dec_scratch = nullptr; c->dec_scratch_floats = 0; }
      DKV_CUDA(c, cudaMalloc(&c->d_dec_scratch, need * sizeof(float)));
      c->dec_scratch_floats = need;
    }
    DecodePtrs ptrs;
    memset(&ptrs, 0, sizeof ptrs);
    for (int i = 0; i < nl; ++i) { ptrs.q[i] = q_dec[l0 + i]; ptrs.kb[i] = kb[l0 + i]; ptrs.vb[i] = vb[l0 + i]; ptrs.out[i] = out[l0 + i]; }
    const dim3 grid(splits, BH, nl);
    const float scale2 = kLog2e / sqrtf((float)s.D);
    ProfScope ps(c, DKV_STEP_DECODE, 1, st);
    if (s.D == 128)
      decode_attend_kernel<128><<<grid, kDecThreads, 0, st>>>(ptrs, layer0 + l0, c->d_held, s.Hkv, s.G, nq, s.L, s.ws, s.rows, scale2,
                                                             c->d_dec_scratch, c->d_dec_tickets + (size_t)(layer0 + l0) * BH);
    else
      decode_attend_kernel<64><<<grid, kDecThreads, 0, st>>>(ptrs, layer0 + l0, c->d_held, s.Hkv, s.G, nq, s.L, s.ws, s.rows, scale2,
                                                            c->d_dec_scratch, c->d_dec_tickets + (size_t)(layer0 + l0) * BH);
    DKV_LAUNCHED(c);
  }
  return DKV_OK;
}

int dkv_get_counts(dkv_ctx* c, int32_t* host_counts, void* stream) {
  if (!c || !host_counts) return DKV_ERR_INVALID_ARG;
  DKV_CUDA(c, cudaMemcpyAsync(host_counts, c->d_count, sizeof(int) * c->s.Bt * c->s.L, cudaMemcpyDeviceToHost,
                              as_stream(stream)));
  DKV_CUDA(c, cudaStreamSynchronize(as_stream(stream)));
  return DKV_OK;
}

int dkv_layer_views(dkv_ctx* c, int32_t layer, const float** scores, const int32_t** idx) {
  int rc = check_layer(c, layer);
  if (rc) return rc;
  if (scores) *scores = c->d_scores + (size_t)layer * layer_scores(c->s);
  if (idx) *idx = c->d_idx + (size_t)layer * layer_idx(c->s);
  return DKV_OK;
}

int dkv_kept_sorted(dkv_ctx* c, int32_t layer, int32_t* sorted_out, void* stream) {
  int rc = check_layer(c, layer);
  if (rc) return rc;
  if (!sorted_out) return DKV_ERR_INVALID_ARG;
  if (!c->gathered[layer]) return DKV_ERR_STATE;
  return do_kept_sorted(c, layer, sorted_out, as_stream(stream));
}

int dkv_budget_views(dkv_ctx* c, const int32_t** cnt, const int32_t** z, const int32_t** zp, const int32_t** held) {
  if (!c) return DKV_ERR_INVALID_ARG;
  const size_t bl = (size_t)c->s.Bt * c->s.L;
  if (cnt) *cnt = c->d_dbg;
  if (z) *z = c->d_dbg + bl;
  if (zp) *zp = c->d_dbg + 2 * bl;
  if (held) *held = c->d_held;
  return DKV_OK;
}

// ---- scoring for callers that cannot allocate ------------------------------------------------------
// Scratch of dkv_score_static: [0, 256) status words, then the partial softmax statistics of
// sweep 1.  The array lives in every GPU that loads the library, from load to exit.  In host code
// its name is only a handle: the device address comes from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_static_scratch[DKV_STATIC_SCRATCH_BYTES];

namespace {
struct StaticSetup { bool done; unsigned char* ptr; int sms; };
StaticSetup g_static_setup[64];
std::mutex g_static_mutex;
}  // namespace

int dkv_score_static(const dkv_config* cfg, const void* q_win, const void* k, float* scores_out, void* stream) {
  int rc = validate(cfg);
  if (rc) return rc;
  if (!q_win || !k || !scores_out || !aligned16(q_win) || !aligned16(k) || !aligned16(scores_out))
    return DKV_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DKV_ERR_CUDA;
  StaticSetup su;
  {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticSetup& g = g_static_setup[dev];
    if (!g.done) {                           // first call on this device
      void* ptr = nullptr;
      if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return DKV_ERR_CUDA;
      int sms = 0;
      if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return DKV_ERR_CUDA;
      if (cudaFuncSetAttribute(tc::score_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes) !=
              cudaSuccess ||
          cudaFuncSetAttribute(tc::score_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes) !=
              cudaSuccess)
        return DKV_ERR_CUDA;
      g.ptr = static_cast<unsigned char*>(ptr);
      g.sms = sms;
      g.done = true;
    }
    su = g;
  }
  const int G = cfg->n_q_heads / cfg->n_kv_heads, heads = cfg->batch * cfg->n_kv_heads;
  const int S = cfg->seq_len, P = S - cfg->window, M = cfg->window * G, D = cfg->head_dim;
  const int tph = (S + tc::kTileKeys - 1) / tc::kTileKeys;
  const long long total_tiles = (long long)heads * tph;
  const int grid = (int)(total_tiles < su.sms ? total_tiles : su.sms);
  int slots = 1;
  for (int bh = 0; bh < heads; ++bh) {
    const int lo = tc::tile_owner((long long)bh * tph, total_tiles, grid);
    const int hi = tc::tile_owner((long long)(bh + 1) * tph - 1, total_tiles, grid);
    if (hi - lo + 1 > slots) slots = hi - lo + 1;
  }
  const unsigned long long need = 256ull + (unsigned long long)heads * slots * 256ull * sizeof(float2);
  if (need > DKV_STATIC_SCRATCH_BYTES) return DKV_ERR_TOO_LARGE;
  cudaStream_t st = as_stream(stream);
  tc::Maps maps;
  memset(&maps, 0, sizeof maps);
  if (!make_map(&maps.q[0], q_win, D, M, heads) || !make_map(&maps.k[0], k, D, S, heads)) return DKV_ERR_CUDA;
  if (cudaMemsetAsync(su.ptr, 0, 256, st) != cudaSuccess) return DKV_ERR_CUDA;   // status words start at zero
  tc::Params p, none;
  memset(&p, 0, sizeof p);
  memset(&none, 0, sizeof none);
  none.mode = tc::kNone;
  p.S = S; p.P = P; p.ws = cfg->window; p.M = M; p.D = D; p.heads = heads; p.half = cfg->pool_kernel / 2;
  p.nl = 1; p.hpl = heads;
  p.back = 0;
  p.wait_cycles = tc::kDefaultWaitCycles;
  p.withhold_tile = -1;
  p.tph = tph; p.nq16 = (M + 15) / 16 * 16; p.nmblk = (M + 127) / 128;
  p.slots = slots; p.m_stride = 256;
  p.scale2 = kLog2e / sqrtf((float)D);
  p.out_scale = (cfg->flags & DKV_F_WINDOW_MEAN) ? 1.0f / (float)M : 1.0f;
  p.pool_avg = cfg->pool_kind == 1;
  p.stats = reinterpret_cast<float2*>(su.ptr + 256);
  p.scores = scores_out; p.copy_out = nullptr;
  p.status = reinterpret_cast<int*>(su.ptr);
  p.stats_grid = grid;
  p.mode = tc::kStats;
  p.idesc = make_idesc(128, 128);
  launch_tc(grid, st, maps, maps, p, none);
  if (cudaGetLastError() != cudaSuccess) return DKV_ERR_CUDA;
  p.mode = tc::kEmit;
  p.idesc = make_idesc(128, p.nq16);
  launch_tc(grid, st, maps, maps, none, p);
  if (cudaGetLastError() != cudaSuccess) return DKV_ERR_CUDA;
  return DKV_OK;
}

int dkv_memcpy_to_host(dkv_ctx* c, void* host_dst, const void* dev_src, uint64_t bytes, void* stream) {
  if (!c || !host_dst || !dev_src) return DKV_ERR_INVALID_ARG;
  DKV_CUDA(c, cudaMemcpyAsync(host_dst, dev_src, bytes, cudaMemcpyDeviceToHost, as_stream(stream)));
  DKV_CUDA(c, cudaStreamSynchronize(as_stream(stream)));
  return DKV_OK;
}

int dkv_last_status(dkv_ctx* c, int32_t* host_status) {
  if (!c || !host_status) return DKV_ERR_INVALID_ARG;
  DKV_CUDA(c, cudaDeviceSynchronize());
  DKV_CUDA(c, cudaMemcpy(host_status, c->d_status, sizeof(int) * 8, cudaMemcpyDeviceToHost));
  if (host_status[0] != 0) DKV_CUDA(c, cudaMemset(c->d_status, 0, sizeof(int) * 8));   // reported once
  host_status[1] = (int32_t)(c->launches & 0x7FFFFFFF);
  return host_status[0] == 0 ? DKV_OK : DKV_ERR_TIMEOUT;
}

int dkv_static_last_status(int32_t* host_status) {
  if (!host_status) return DKV_ERR_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess) return DKV_ERR_CUDA;
  if (cudaMemcpyFromSymbol(host_status, g_static_scratch, sizeof(int) * 8) != cudaSuccess) return DKV_ERR_CUDA;
  host_status[1] = 0;
  return host_status[0] == 0 ? DKV_OK : DKV_ERR_TIMEOUT;
}

int dkv_set_wait_limit(dkv_ctx* c, int64_t clock_ticks) {
  if (!c || clock_ticks < 1000) return DKV_ERR_INVALID_ARG;
  c->wait_cycles = clock_ticks;
  if (c->pass_exec) { cudaGraphExecDestroy(c->pass_exec); c->pass_exec = nullptr; }   // recorded with the old limit
  return DKV_OK;
}

int dkv_debug_withhold_tile(dkv_ctx* c, int32_t sweep, int32_t tile) {
  if (!c || (tile >= 0 && sweep != 1 && sweep != 2)) return DKV_ERR_INVALID_ARG;
  c->withhold_sweep = tile >= 0 ? sweep : -1;
  c->withhold_tile = tile >= 0 ? tile : -1;
  if (c->pass_exec) { cudaGraphExecDestroy(c->pass_exec); c->pass_exec = nullptr; }
  return DKV_OK;
}

int dkv_profile(dkv_ctx* c, int enable) {
  if (!c) return DKV_ERR_INVALID_ARG;
  c->prof_on = enable != 0;
  return DKV_OK;
}

int dkv_profile_read(dkv_ctx* c, double* ms, int64_t* launches) {
  if (!c || !ms || !launches) return DKV_ERR_INVALID_ARG;
  DKV_CUDA(c, cudaDeviceSynchronize());
  for (size_t i = 0; i < c->prof_used; ++i) {
    const ProfRec& r = (*c->prof_recs)[i];
    float t = 0.f;
    if (cudaEventElapsedTime(&t, r.a, r.b) == cudaSuccess) {
      c->prof_ms[r.step] += t;
      c->prof_launches[r.step] += r.launches;
    }
  }
  c->prof_used = 0;
  for (int i = 0; i < DKV_N_STEPS; ++i) {
    ms[i] = c->prof_ms[i]; launches[i] = c->prof_launches[i];
    c->prof_ms[i] = 0; c->prof_launches[i] = 0;
  }
  return DKV_OK;
}

int64_t dkv_launch_count(dkv_ctx* c) { return c ? (int64_t)c->launches : -1; }

int dkv_last_cuda_error(dkv_ctx* c) { return c ? c->last_cuda : 0; }

}  // extern "C"
