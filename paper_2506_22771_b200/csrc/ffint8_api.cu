// C ABI of libffint8 (declared in include/ffint8.h): host-side validation, launch sequencing of
// the per-layer FF-INT8 step (Sec. IV-B, Fig. 4) and of Algorithm 1's epoch body.
#include "../../include/ffint8.h"

#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <type_traits>
#include <vector>

#include "common.cuh"
#include "elementwise.cuh"
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "dwconv.cuh"
#include "conv_small.cuh"

using namespace ffi8;

struct ff_ctx {
  int device = 0;
  int sm_count = 148;
  void* workspace = nullptr;
  size_t workspace_bytes = 0;
  bool status_zeroed = false;
  int gemm_path = FF_GEMM_AUTO;
  uint64_t launches = 0;
  TcState tc;
  // optional per-kernel timing (ff_profile_start / ff_profile_stop)
  bool profiling = false;
  struct ProfRec {
    int kid;
    cudaEvent_t a, b;
  };
  std::vector<ProfRec> prof_recs;
  std::vector<cudaEvent_t> prof_pool;
  // set for the duration of a data-parallel phase call: the 2B rows at hand are rows [row_off, row_off + B)
  // of each set of a batch of B_total rows per set (B_total == 0: the batch is not split)
  struct Shard {
    int B_total = 0;
    int row_off = 0;
    int B_local = 0;
  } shard;
  bool accumulate_only = false;  // weight-gradient contractions leave their INT32 sums in accW_dump, no update
  bool joint_range = false;      // the two halves of the batch are quantised with one range (classification: the halves
                                 // are groups of candidate labels, not a positive and a negative set)
  // captured launch sequences of ff_train_step (ff_set_graph_mode)
  bool graph_mode = false;
  struct GraphEntry {
    std::vector<unsigned char> key;  // everything the launch sequence depends on, compared byte by byte
    cudaGraphExec_t exec = nullptr;
    uint64_t launches = 0;           // kernel launches one replay stands for
    bool eager_only = false;         // capture failed once: this call shape stays on the eager path
    uint64_t last_use = 0;
  };
  std::vector<GraphEntry> graphs;
  uint64_t graph_clock = 0;
  uint64_t graph_replays = 0;
  cudaStream_t capture_stream = nullptr;  // captures are recorded here (the caller's may be the legacy stream, which cannot capture)
  char err[512] = {0};
};

namespace {

// workspace layout: [0, 256) status word (+ padding), then the loss kernel's partial-sum scratch
constexpr size_t WS_STATUS_BYTES = 256;
constexpr size_t WS_STEP_OFFSET = 64;   // StepState inside the status block
constexpr size_t WS_LOSS_OFFSET = WS_STATUS_BYTES;
// one scratch per layer: the losses of all layers of a step are computed by one launch
constexpr size_t WS_BYTES = (WS_LOSS_OFFSET + (FF_MAX_LATER + 1) * sizeof(LossScratch) + 255) / 256 * 256;  // fixed header
// After the header: INT32 partial-sum slabs of a split weight-gradient contraction,
// [splits][2 sets][N][K].  Splitting is used where the output N x K alone has too few tiles to
// occupy the device (convolutions contract over every output position of the batch).
constexpr size_t WS_SLAB_CAP = (size_t)64 << 20;  // never ask for more than this per layer
constexpr int WS_TARGET_ITEMS = 296;               // tiles x splits aimed at (two per SM of a 148-SM device)

ff_status fail(ff_ctx* ctx, ff_status st, const char* fmt, const char* a = "", long long b = 0) {
  if (ctx) snprintf(ctx->err, sizeof(ctx->err), fmt, a, b);
  return st;
}

#define FF_CUDA(ctx, call)                                                                  \
  do {                                                                                      \
    cudaError_t e__ = (call);                                                               \
    if (e__ != cudaSuccess) return fail(ctx, FF_ERR_CUDA, "%s (line %lld)", cudaGetErrorString(e__), __LINE__); \
  } while (0)

#define FF_LAUNCH_CHECK(ctx)                                                                \
  do {                                                                                      \
    (ctx)->launches++;                                                                      \
    cudaError_t e__ = cudaGetLastError();                                                   \
    if (e__ != cudaSuccess) return fail(ctx, FF_ERR_CUDA, "launch: %s (line %lld)", cudaGetErrorString(e__), __LINE__); \
  } while (0)

// CUDA-event pair around one kernel launch while profiling is on (events come from a pool that grows
// on the host only; nothing is allocated on the device).
struct ProfScope {
  ff_ctx* ctx;
  cudaStream_t st;
  cudaEvent_t b = nullptr;
  ProfScope(ff_ctx* c, int kid, cudaStream_t s) : ctx(c), st(s) {
    if (!c->profiling) return;
    cudaEvent_t ev[2] = {nullptr, nullptr};
    for (auto& e : ev) {
      if (!c->prof_pool.empty()) {
        e = c->prof_pool.back();
        c->prof_pool.pop_back();
      } else if (cudaEventCreate(&e) != cudaSuccess) {
        e = nullptr;
      }
    }
    if (!ev[0] || !ev[1]) return;
    cudaEventRecord(ev[0], s);
    b = ev[1];
    c->prof_recs.push_back({kid, ev[0], ev[1]});
  }
  ~ProfScope() {
    if (b) cudaEventRecord(b, st);
  }
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// output rows (positions) per sample, and input rows per sample (they differ for a strided convolution)
inline int rows_per_sample(const ff_layer_desc& L) { return L.kind != FF_LINEAR ? tc_out_h(L) * tc_out_w(L) : 1; }
// values per sample of what the layer hands to the next one (a quarter of the positions with 2x2 pooling)
inline long long next_values_per_sample(const ff_layer_desc& L) {
  return (long long)rows_per_sample(L) / (L.pool == 2 ? 4 : 1) * L.N;
}
inline int in_rows_per_sample(const ff_layer_desc& L) { return L.kind != FF_LINEAR ? L.H * L.Wd : 1; }
inline int in_features(const ff_layer_desc& L) { return (L.kind == FF_CONV3X3 || L.kind == FF_DWCONV3X3) ? L.Cin : L.K; }

ff_status check_layer(ff_ctx* ctx, const ff_layer_desc* L, int B) {
  if (!L) return fail(ctx, FF_ERR_ARG, "layer descriptor is NULL");
  if (B <= 0) return fail(ctx, FF_ERR_ARG, "B must be positive");
  if (L->kind != FF_LINEAR && L->kind != FF_CONV3X3 && L->kind != FF_CONV1X1 && L->kind != FF_DWCONV3X3)
    return fail(ctx, FF_ERR_ARG, "unknown layer kind");
  if (L->kind == FF_DWCONV3X3 && (L->H <= 0 || L->Wd <= 0 || L->Cin <= 0 || L->N != L->Cin || L->K != 9))
    return fail(ctx, FF_ERR_ARG, "dwconv3x3 needs H, Wd, Cin > 0, N = Cin and K = 9");
  if (L->kind == FF_CONV1X1 && (L->H <= 0 || L->Wd <= 0 || L->Cin <= 0 || L->K != L->Cin))
    return fail(ctx, FF_ERR_ARG, "conv1x1 needs H, Wd, Cin > 0 and K = Cin");
  if (L->K <= 0 || L->N <= 0) return fail(ctx, FF_ERR_ARG, "K and N must be positive");
  if (L->kind == FF_CONV3X3 && (L->H <= 0 || L->Wd <= 0 || L->Cin <= 0 || L->K != 9 * L->Cin))
    return fail(ctx, FF_ERR_ARG, "conv3x3 needs H, Wd, Cin > 0 and K = 9*Cin");
  if (L->stride < 0 || L->stride > 2 || (L->stride == 2 && L->kind != FF_CONV3X3 && L->kind != FF_DWCONV3X3))
    return fail(ctx, FF_ERR_ARG, "stride must be 0 / 1, or 2 for a conv3x3 / dwconv3x3 layer");
  for (int r : {L->round_x, L->round_w, L->round_dh})
    if (r != FF_ROUND_NEAREST_EVEN && r != FF_ROUND_STOCHASTIC) return fail(ctx, FF_ERR_ARG, "unknown rounding mode");
  if (!(L->eps > 0.0f)) return fail(ctx, FF_ERR_ARG, "eps must be > 0");
  if (!(L->momentum >= 0.0f && L->momentum < 1.0f)) return fail(ctx, FF_ERR_ARG, "momentum must lie in [0, 1)");
  if (L->pool < 0 || L->pool > 2) return fail(ctx, FF_ERR_ARG, "pool must be 0, 1 or 2");
  if (L->pool == 2 && (L->kind == FF_LINEAR || tc_out_h(*L) % 2 || tc_out_w(*L) % 2))
    return fail(ctx, FF_ERR_ARG, "pooling needs a spatial layer with even output extents");
  if (L->optimizer != FF_OPT_SGD && L->optimizer != FF_OPT_ADAM) return fail(ctx, FF_ERR_ARG, "unknown optimizer");
  if (L->optimizer == FF_OPT_ADAM && (!(L->beta2 >= 0.0f && L->beta2 < 1.0f) || !(L->adam_eps >= 0.0f)))
    return fail(ctx, FF_ERR_ARG, "Adam needs beta2 in [0, 1) and adam_eps >= 0");
  const long long R = rows_per_sample(*L);
  const long long rows = 2LL * B * R;
  // 32-bit rounding counters and element indices
  const long long rows_in = 2LL * B * in_rows_per_sample(*L);
  if (rows * L->N >= (1LL << 32) || rows_in * in_features(*L) >= (1LL << 32) || (long long)L->N * L->K >= (1LL << 32))
    return fail(ctx, FF_ERR_RANGE, "tensor has 2^32 or more elements");
  if (rows >= (1LL << 31)) return fail(ctx, FF_ERR_RANGE, "too many rows");
  // worst-case INT32 accumulator range: 127*127*contraction length < 2^31  (Sec. IV-B: INT32 accumulation)
  const long long lim = ((1LL << 31) - 1) / (127LL * 127LL);
  if (L->K > lim) return fail(ctx, FF_ERR_RANGE, "forward contraction %s%lld too long for INT32", "", L->K);
  if (L->kind == FF_LINEAR && (long long)B * R > lim)
    return fail(ctx, FF_ERR_RANGE, "weight-gradient contraction %s%lld too long for INT32", "", (long long)B * R);
  return FF_OK;
}

ff_status check_bufs(ff_ctx* ctx, const ff_layer_bufs* b, bool need_x) {
  if (!b) return fail(ctx, FF_ERR_ARG, "buffer struct is NULL");
  const void* req[] = {b->W, b->Y, b->G, b->Xq, b->Wq, b->dHq, b->absmax, b->S, b->rowmax, b->coef, b->loss};
  for (const void* p : req)
    if (!p) return fail(ctx, FF_ERR_ARG, "a required device pointer is NULL");
  if (need_x && !b->X) return fail(ctx, FF_ERR_ARG, "X is NULL");
  const void* all[] = {b->W, b->X, b->Y, b->G, b->Xnext, b->Xq, b->Wq, b->dHq, b->absmax, b->S, b->rowmax, b->coef,
                       b->loss, b->acc_dump, b->accW_dump, b->Mom, b->Var, b->Skip};
  for (const void* p : all)
    if (p && !aligned16(p)) return fail(ctx, FF_ERR_ALIGN, "a device pointer is not 16-byte aligned");
  if (b->Skip && (!b->Xnext || b->Skip == b->Xnext)) return fail(ctx, FF_ERR_ARG, "a skip path needs Xnext, distinct from Skip");
  return FF_OK;
}

// Row pitches of the INT8 tensors: linear layers only, at least the row length, multiples of 16 bytes.
ff_status check_pitches(ff_ctx* ctx, const ff_layer_desc* L, const ff_layer_bufs* b) {
  if (b->Skip && L->pool == 2) return fail(ctx, FF_ERR_ARG, "a pooled output takes no skip path");
  if (!b->ld_xq && !b->ld_dhq) return FF_OK;
  if (L->kind != FF_LINEAR) return fail(ctx, FF_ERR_ARG, "row pitches are for linear layers only");
  if (b->ld_xq && (b->ld_xq < L->K || b->ld_xq % 16)) return fail(ctx, FF_ERR_ARG, "ld_xq must be >= K and a multiple of 16");
  if (b->ld_dhq && (b->ld_dhq < L->N || b->ld_dhq % 16)) return fail(ctx, FF_ERR_ARG, "ld_dhq must be >= N and a multiple of 16");
  return FF_OK;
}

ff_status check_ctx(ff_ctx* ctx) {
  if (!ctx) return FF_ERR_ARG;
  if (!ctx->workspace) return fail(ctx, FF_ERR_WORKSPACE, "no workspace set");
  return FF_OK;
}

inline uint32_t* status_ptr(ff_ctx* ctx) { return reinterpret_cast<uint32_t*>(ctx->workspace); }
// Per-sample normalisation factors of the layer whose forward has just run ([2B] floats at the start of the
// transient region: written by the goodness finalisation, read by the normalisation pass that follows it, before
// anything else uses the region); NULL when the workspace has no room, the pass then forms them itself.
inline float* factors_ptr(ff_ctx* ctx, int B) {
  if (ctx->workspace_bytes < WS_BYTES + (size_t)2 * B * sizeof(float)) return nullptr;
  return reinterpret_cast<float*>(static_cast<char*>(ctx->workspace) + WS_BYTES);
}
inline StepState* step_ptr(ff_ctx* ctx) {
  return reinterpret_cast<StepState*>(static_cast<char*>(ctx->workspace) + WS_STEP_OFFSET);
}
// Publishes the step counter (and lambda) to the kernels of the calls that follow on `st`.
// With a layer list, the range vectors of those layers are cleared by the same launch (a whole-network call starts
// by taking ranges; the launch is issued outside any captured sequence, so it costs the replayed step nothing).
ff_status set_step(ff_ctx* ctx, uint64_t step, float lambda, bool with_lambda, cudaStream_t st,
                   const ff_layer_bufs* bufs = nullptr, int n_layers = 0) {
  static_assert(FF_MAX_LATER + 1 <= 32 && FF_ABSMAX_LEN == 8, "RangeTable holds 32 vectors of 8 floats");
  RangeTable rt;
  rt.n = bufs ? n_layers : 0;
  for (int l = 0; l < rt.n; ++l) rt.p[l] = bufs[l].absmax;
  set_step_kernel<<<1, 256, 0, st>>>(step_ptr(ctx), step, lambda, with_lambda ? 1 : 0, rt);
  FF_LAUNCH_CHECK(ctx);
  return FF_OK;
}

ff_status ensure_status(ff_ctx* ctx, cudaStream_t st) {
  if (!ctx->status_zeroed) {
    FF_CUDA(ctx, cudaMemsetAsync(ctx->workspace, 0, WS_BYTES, st));  // status word and the loss kernel's ticket
    ctx->status_zeroed = true;
  }
  return FF_OK;
}

// Offsets that turn a shard's local element index into the index in the unsplit [2][B_total][per_sample]
// tensor (the stochastic-rounding counter), for the positive and the negative pass.
inline uint2 ctr_bias(const ff_ctx* ctx, size_t per_sample, int B) {
  if (!ctx->shard.B_total) return uint2{0u, 0u};
  const uint32_t off = (uint32_t)((size_t)ctx->shard.row_off * per_sample);
  return uint2{off, (uint32_t)((size_t)(ctx->shard.B_total - B) * per_sample) + off};
}

inline int ew_blocks(ff_ctx* ctx, size_t work_items, int per_thread = 4) {
  size_t need = (work_items + (size_t)EW_THREADS * per_thread - 1) / ((size_t)EW_THREADS * per_thread);
  size_t cap = (size_t)ctx->sm_count * 8;
  size_t b = need < cap ? need : cap;
  return (int)(b ? b : 1);
}

// ---- contraction dispatch ----------------------------------------------------------------
template <class LA, class LB, bool TRANS, int NPASS, class Epi>
ff_status launch_simt(ff_ctx* ctx, LA la, LB lb, int out_rows, int out_cols, int clen, Epi epi, cudaStream_t st,
                      int splits = 1) {
  // contraction elements per split, a multiple of the kernel's contraction block
  const int csplit = splits > 1 ? ((clen + splits - 1) / splits + SG_BK - 1) / SG_BK * SG_BK : clen;
  dim3 grid((out_cols + SG_BN - 1) / SG_BN, (out_rows + SG_BM - 1) / SG_BM, splits > 1 ? (clen + csplit - 1) / csplit : 1);
  ProfScope prof(ctx, std::is_same<Epi, ForwardEpilogue>::value ? FF_K_FWD_GEMM : std::is_same<Epi, UpdateEpilogue>::value ? FF_K_UPD_GEMM : FF_K_RAW_GEMM, st);
  gemm_simt_kernel<LA, LB, TRANS, NPASS, Epi><<<grid, SG_THREADS, 0, st>>>(la, lb, clen, csplit, epi);
  FF_LAUNCH_CHECK(ctx);
  return FF_OK;
}

inline DenseView dense(const int8_t* p, int rows, int cols, int ld = 0) {
  if (!ld) ld = cols;
  return DenseView{p, rows, cols, ld, (cols % 8 == 0) && (ld % 8 == 0) && ((reinterpret_cast<uintptr_t>(p) & 7) == 0)};
}
// row padding of a dense layer's INT8 tensor with `cols` values per row and a pitch of ld bytes (0: none)
inline RowPad row_pad(int cols, int ld) { return RowPad{(uint32_t)cols, ld ? (uint32_t)(ld - cols) : 0u}; }
inline Im2colView im2col(const int8_t* p, const ff_layer_desc& L, int samples) {
  return Im2colView{p, samples * tc_out_h(L) * tc_out_w(L), 9 * L.Cin, L.H, L.Wd, L.Cin, tc_out_h(L), tc_out_w(L),
                    tc_conv_stride(L), (L.Cin % 8 == 0) && ((reinterpret_cast<uintptr_t>(p) & 7) == 0)};
}

// ---- split weight gradient ------------------------------------------------------------------
inline long long simt_tiles(const ff_layer_desc& L) {
  return (long long)((L.N + SG_BM - 1) / SG_BM) * ((L.K + SG_BN - 1) / SG_BN);
}
// Number of splits the SIMT weight gradient asks for (1 = none): enough that tiles x splits reaches
// WS_TARGET_ITEMS, at least 1024 contraction elements per split, slabs within WS_SLAB_CAP and within
// the workspace actually set (`ws_bytes`; pass SIZE_MAX to get the wish) - but never fewer than keep every
// split's contraction within WG_SAFE_LEN, so that no INT32 partial sum can wrap (simt_min_splits; the caller
// refuses a workspace too small for that many).
inline int simt_min_splits(const ff_layer_desc& L, int B) {
  const long long clen = (long long)B * rows_per_sample(L);
  const long long safe = WG_SAFE_LEN / SG_BK * SG_BK;  // a split's length is rounded up to contraction blocks
  return (int)((clen + safe - 1) / safe);
}
// One shard of a split batch whose WHOLE contraction can leave INT32: its local sums must pass through the update
// kernel's range check (a share of the range per shard), so the routes that would write them straight to accW_dump
// take at least two splits.
inline bool dp_checks_needed(const ff_ctx* ctx, const ff_layer_desc& L) {
  return ctx->shard.B_total > 0 && (long long)ctx->shard.B_total * rows_per_sample(L) > WG_SAFE_LEN;
}
inline int simt_wgrad_splits(const ff_layer_desc& L, int B, size_t ws_bytes) {
  const long long clen = (long long)B * rows_per_sample(L);
  const long long tiles = simt_tiles(L);
  long long splits = (WS_TARGET_ITEMS + tiles - 1) / tiles;
  if (splits > clen / 1024) splits = clen / 1024;
  const size_t per_split = (size_t)2 * L.N * L.K * sizeof(int32_t);
  const size_t room = ws_bytes > WS_BYTES ? ws_bytes - WS_BYTES : 0;
  const int need = simt_min_splits(L, B);
  if ((size_t)splits * per_split > WS_SLAB_CAP) splits = (long long)(WS_SLAB_CAP / per_split);
  if (splits < need) splits = need;
  if ((size_t)splits * per_split > room) splits = (long long)(room / per_split);
  return splits < 2 ? 1 : (int)splits;
}
// grid.z the split launch really uses (the last splits can be empty after rounding to blocks)
inline int simt_split_count(int clen, int splits) {
  const int csplit = ((clen + splits - 1) / splits + SG_BK - 1) / SG_BK * SG_BK;
  return (clen + csplit - 1) / csplit;
}

ff_status launch_slab_update(ff_ctx* ctx, const int32_t* slabs, int splits, const ff_layer_desc& L, const ff_layer_bufs& b,
                             cudaStream_t st, int pitch = 0) {
  const size_t plane = (size_t)L.N * L.K;
  float* W = ctx->accumulate_only ? nullptr : b.W;
  int32_t* dump = b.accW_dump == slabs ? nullptr : b.accW_dump;  // the sums already are where they would be copied to
  UpdateRule rule;
  rule.kind = L.optimizer == FF_OPT_ADAM ? 1 : 0;
  rule.lr = L.lr, rule.mu = L.momentum, rule.beta2 = L.beta2, rule.eps = L.adam_eps;
  rule.Mom = (rule.kind == 1 || L.momentum != 0.0f) ? b.Mom : nullptr;
  rule.Var = rule.kind == 1 ? b.Var : nullptr;
  rule.ss = step_ptr(ctx);
  if (!W && !dump) return FF_OK;
  // Largest magnitude a sum may have.  One shard of a split batch: its share of the INT32 range in proportion to
  // its rows, so that the sums of all shards cannot wrap when the caller adds them in 32 bits (sufficient, not
  // necessary: a shard may be refused although the whole batch would have fitted).
  long long limit = 2147483647LL;
  if (ctx->accumulate_only && ctx->shard.B_total > 0)
    limit = limit / ctx->shard.B_total * ctx->shard.B_local;
  if (splits <= 2 && (pitch == 0 || pitch == L.K) && (plane & 3) == 0 && plane >= ((size_t)1 << 18)) {
    const size_t want = (plane / 4 + 255) / 256, cap = (size_t)ctx->sm_count * 8;
    slab_update_flat_kernel<<<(unsigned)(want < cap ? want : cap), 256, 0, st>>>(slabs, splits, plane, W, b.absmax, rule, dump, limit,
                                                                                 status_ptr(ctx));
  } else {
    const size_t want = (plane + 31) / 32, cap = (size_t)ctx->sm_count * 8;
    slab_update_kernel<<<(unsigned)(want < cap ? want : cap), 256, 0, st>>>(slabs, splits, plane, L.K, pitch ? pitch : L.K, W,
                                                                            b.absmax, rule, dump, limit, status_ptr(ctx));
  }
  FF_LAUNCH_CHECK(ctx);
  return FF_OK;
}

// ---- explicit-im2col route for convolutions with few input channels -------------------------
// Transient workspace after the header: [ xi: rows x kpad | wi: N x kpad | slabs ], each 256-byte aligned.
struct Im2colPlan {
  int kpad;
  size_t xi_off, wi_off, slab_off, slab_bytes_per_split;
  int max_splits;   // that fit the workspace (the wish when ws_bytes = SIZE_MAX); -1: xi / wi do not fit
};
inline size_t up256(size_t v) { return (v + 255) / 256 * 256; }
inline Im2colPlan im2col_plan(const ff_layer_desc& L, int B, size_t ws_bytes, int sm_count) {
  Im2colPlan pl;
  pl.kpad = tc_im2col_kpad(L);
  const size_t rows = (size_t)2 * B * tc_out_h(L) * tc_out_w(L);
  pl.xi_off = WS_BYTES;
  pl.wi_off = pl.xi_off + up256(rows * pl.kpad);
  pl.slab_off = pl.wi_off + up256((size_t)L.N * pl.kpad);
  pl.slab_bytes_per_split = (size_t)2 * L.N * pl.kpad * sizeof(int32_t);
  const int wish = tc_dense_slab_splits(L.N, pl.kpad, (long long)B * tc_out_h(L) * tc_out_w(L), sm_count);
  const size_t room = ws_bytes > pl.slab_off ? ws_bytes - pl.slab_off : 0;
  const size_t fit = room / pl.slab_bytes_per_split;
  pl.max_splits = ws_bytes < pl.slab_off ? -1 : (int)(fit < (size_t)wish ? fit : (size_t)wish);
  return pl;
}
inline bool im2col_route(ff_ctx* ctx, const ff_layer_desc& L, int B) {
  if (ctx->gemm_path == FF_GEMM_SIMT || !tc_im2col_ok(L)) return false;
  // room for xi / wi and for as many slabs as keep every split's contraction within WG_SAFE_LEN
  const int need = tc_min_splits(((long long)B * tc_out_h(L) * tc_out_w(L) + 127) / 128);
  return im2col_plan(L, B, ctx->workspace_bytes, ctx->sm_count).max_splits >= need;
}
// Writes xi (and wi) for layer L from its Xq (and Wq).
ff_status launch_im2col(ff_ctx* ctx, const ff_layer_desc& L, const ff_layer_bufs& b, int B, const Im2colPlan& pl, bool weights,
                        cudaStream_t st) {
  char* ws = static_cast<char*>(ctx->workspace);
  int8_t* xi = reinterpret_cast<int8_t*>(ws + pl.xi_off);
  const int Ho = tc_out_h(L), Wo = tc_out_w(L), sd = tc_conv_stride(L);
  const int rows = 2 * B * Ho * Wo;
  const int blocks = (rows + 255) / 256;
  switch (pl.kpad) {
    case 16: im2col3x3_kernel<16><<<blocks, 256, 0, st>>>(b.Xq, xi, rows, L.H, L.Wd, L.Cin, Ho, Wo, sd); break;
    case 32: im2col3x3_kernel<32><<<blocks, 256, 0, st>>>(b.Xq, xi, rows, L.H, L.Wd, L.Cin, Ho, Wo, sd); break;
    case 48: im2col3x3_kernel<48><<<blocks, 256, 0, st>>>(b.Xq, xi, rows, L.H, L.Wd, L.Cin, Ho, Wo, sd); break;
    case 64: im2col3x3_kernel<64><<<blocks, 256, 0, st>>>(b.Xq, xi, rows, L.H, L.Wd, L.Cin, Ho, Wo, sd); break;
    case 96: im2col3x3_kernel<96><<<blocks, 256, 0, st>>>(b.Xq, xi, rows, L.H, L.Wd, L.Cin, Ho, Wo, sd); break;
    default: im2col3x3_kernel<128><<<blocks, 256, 0, st>>>(b.Xq, xi, rows, L.H, L.Wd, L.Cin, Ho, Wo, sd); break;
  }
  FF_LAUNCH_CHECK(ctx);
  if (weights) {
    int8_t* wi = reinterpret_cast<int8_t*>(ws + pl.wi_off);
    pad_rows_kernel<<<(L.N * pl.kpad + 255) / 256, 256, 0, st>>>(b.Wq, wi, L.N, L.K, pl.kpad);
    FF_LAUNCH_CHECK(ctx);
  }
  return FF_OK;
}

// Forward contraction + fused epilogue.
// ---- depthwise layers: streaming kernels of their own (no contraction) ------------------------------
inline DwGeom dw_geom(const ff_layer_desc& L, int B) {
  DwGeom g;
  g.H = L.H, g.W = L.Wd, g.C = L.Cin, g.Ho = tc_out_h(L), g.Wo = tc_out_w(L), g.stride = tc_conv_stride(L);
  g.rows_per_sample = g.Ho * g.Wo;
  g.rows_per_pass = B * g.rows_per_sample;
  g.rows = 2 * g.rows_per_pass;
  g.imgs_per_pass = B;
  g.wblocks = (g.Wo + DW_WB - 1) / DW_WB;
  return g;
}
// four channels per thread need whole words; the per-channel weight table must fit the default shared memory
inline bool dw_vec(const ff_layer_desc& L) { return L.Cin % 4 == 0 && (size_t)L.Cin * 36 <= 40 * 1024; }

ff_status dw_forward(ff_ctx* ctx, const ff_layer_desc& L, const ff_layer_bufs& b, int B, cudaStream_t st) {
  const DwGeom g = dw_geom(L, B);
  ProfScope prof(ctx, FF_K_DW_FWD, st);
  unsigned long long* S = reinterpret_cast<unsigned long long*>(b.S);
  if (dw_vec(L)) {
    const size_t items = (size_t)2 * B * g.Ho * g.wblocks * (g.C / 4);
    const int grid = ew_blocks(ctx, items, 1);
    if (g.stride == 2)
      dwconv3x3_fwd_kernel<2><<<grid, DW_THREADS, (size_t)g.C * 36, st>>>(b.Xq, b.Wq, b.Y, b.acc_dump, S, b.rowmax, b.absmax, g);
    else
      dwconv3x3_fwd_kernel<1><<<grid, DW_THREADS, (size_t)g.C * 36, st>>>(b.Xq, b.Wq, b.Y, b.acc_dump, S, b.rowmax, b.absmax, g);
  } else {
    const int grid = ew_blocks(ctx, (size_t)g.rows * g.C, 1);
    dwconv3x3_fwd_scalar_kernel<<<grid, DW_THREADS, 0, st>>>(b.Xq, b.Wq, b.Y, b.acc_dump, S, b.rowmax, b.absmax, g);
  }
  FF_LAUNCH_CHECK(ctx);
  return FF_OK;
}

// Planes of INT32 sums a depthwise layer keeps room for ([plane][2][C][9]).  No plane sums over more than
// WG_SAFE_LEN positions of a set; a plane holds whole chunks of positions, and a chunk is at most half that
// long, so every plane but the last is at least half full: twice the minimum, plus one, always suffices.
inline int dw_planes(const ff_layer_desc& L, int B) {
  const long long padded = (long long)B * tc_out_h(L) * ((tc_out_w(L) + DW_WB - 1) / DW_WB) * DW_WB;
  return 2 * (int)((padded + WG_SAFE_LEN - 1) / WG_SAFE_LEN) + 1;
}
// INT32 sums of both sets into the workspace ([plane][2][C][9], cleared first), then the common reduce / update kernel.
ff_status dw_update(ff_ctx* ctx, const ff_layer_desc& L, const ff_layer_bufs& b, int B, cudaStream_t st) {
  const DwGeom g = dw_geom(L, B);
  const size_t plane_bytes = (size_t)2 * g.C * 9 * sizeof(int32_t);
  const size_t bytes = plane_bytes * dw_planes(L, B);
  if (ctx->workspace_bytes < WS_BYTES + bytes)
    return fail(ctx, FF_ERR_WORKSPACE, "workspace has no room for the depthwise weight-gradient sums");
  int32_t* accW = reinterpret_cast<int32_t*>(static_cast<char*>(ctx->workspace) + WS_BYTES);
  ProfScope prof(ctx, FF_K_DW_UPD, st);
  const bool was = ctx->profiling;
  ctx->profiling = false;  // one event pair around the whole route
  cudaError_t e = cudaMemsetAsync(accW, 0, bytes, st);
  if (e != cudaSuccess) {
    ctx->profiling = was;
    return fail(ctx, FF_ERR_CUDA, "%s", cudaGetErrorString(e));
  }
  int planes = 1;
  const bool vec = L.Cin % 4 == 0;
  const int tiles = vec ? (g.C / 4 + 31) / 32 : 1;
  // units of the contraction a block strides through: position blocks of DW_WB outputs (vector form) or positions
  const int units = vec ? B * g.Ho * g.wblocks : g.rows_per_pass;
  const long long safe_units = vec ? WG_SAFE_LEN / DW_WB : WG_SAFE_LEN, half_units = safe_units / 2;
  // enough chunks to occupy the device several times over, not shorter than 32 (64) units - and none longer than
  // half of what a plane may sum over
  int chunks = vec ? (ctx->sm_count * 8 + 2 * tiles - 1) / (2 * tiles) : ctx->sm_count * 4;
  const int max_chunks = vec ? (units + 31) / 32 : (units + 63) / 64;
  if (chunks > max_chunks) chunks = max_chunks;
  if (chunks < (units + half_units - 1) / half_units) chunks = (int)((units + half_units - 1) / half_units);
  const int per = (units + chunks - 1) / chunks;
  const int bpp = (int)(safe_units / per);   // chunks that share a plane (>= 2)
  const dim3 grid((units + per - 1) / per, tiles, 2);
  planes = ((int)grid.x + bpp - 1) / bpp;
  if (planes > dw_planes(L, B)) {
    ctx->profiling = was;
    return fail(ctx, FF_ERR_WORKSPACE, "depthwise weight gradient: more planes than planned");
  }
  if (vec && g.stride == 2)
    dwconv3x3_wgrad_kernel<2><<<grid, DW_THREADS, 0, st>>>(b.dHq, b.Xq, accW, g, per, bpp);
  else if (vec)
    dwconv3x3_wgrad_kernel<1><<<grid, DW_THREADS, 0, st>>>(b.dHq, b.Xq, accW, g, per, bpp);
  else
    dwconv3x3_wgrad_scalar_kernel<<<grid, DW_THREADS, 0, st>>>(b.dHq, b.Xq, accW, g, per, bpp);
  ctx->launches++;
  ff_status s = FF_OK;
  if ((e = cudaGetLastError()) != cudaSuccess) s = fail(ctx, FF_ERR_CUDA, "launch: %s", cudaGetErrorString(e));
  if (s == FF_OK) s = launch_slab_update(ctx, accW, planes, L, b, st, 0);
  ctx->profiling = was;
  return s;
}

// 3x3 convolution with at most four input channels: direct dp4a kernel (conv_small.cuh)
ff_status conv_small_forward(ff_ctx* ctx, const ff_layer_desc& L, const ff_layer_bufs& b, int B, cudaStream_t st) {
  ConvSmallGeom g;
  g.H = L.H, g.W = L.Wd, g.Ho = tc_out_h(L), g.Wo = tc_out_w(L), g.stride = tc_conv_stride(L), g.N = L.N;
  g.rows_per_sample = g.Ho * g.Wo;
  g.rows_per_pass = B * g.rows_per_sample;
  g.rows = 2 * g.rows_per_pass;
  g.y_stream = (size_t)g.rows * L.N * sizeof(float) > ((size_t)80 << 20) ? 1 : 0;
  const int tiles = (g.rows + CS_THREADS - 1) / CS_THREADS;
  const int cap = ctx->sm_count * 4;
  const int grid = tiles < cap ? tiles : cap;
  unsigned long long* S = reinterpret_cast<unsigned long long*>(b.S);
  ProfScope prof(ctx, FF_K_FWD_GEMM, st);
#define FF_CS_LAUNCH(CIN, NN) \
  conv3x3_small_fwd_kernel<CIN, NN><<<grid, CS_THREADS, 0, st>>>(b.Xq, b.Wq, b.Y, b.acc_dump, S, b.rowmax, b.absmax, g)
#define FF_CS_BY_N(CIN)                    \
  switch (L.N) {                           \
    case 16: FF_CS_LAUNCH(CIN, 16); break;  \
    case 32: FF_CS_LAUNCH(CIN, 32); break;  \
    case 64: FF_CS_LAUNCH(CIN, 64); break;  \
    default: FF_CS_LAUNCH(CIN, 128); break; \
  }
  switch (L.Cin) {
    case 1: FF_CS_BY_N(1); break;
    case 2: FF_CS_BY_N(2); break;
    case 3: FF_CS_BY_N(3); break;
    default: FF_CS_BY_N(4); break;
  }
#undef FF_CS_BY_N
#undef FF_CS_LAUNCH
  FF_LAUNCH_CHECK(ctx);
  return FF_OK;
}

// Weight gradient of the same layers: direct dp4a kernel into (slab, set) planes of INT32 sums, then the common
// reduce + update kernel (which also checks the INT32 range of the whole sums).
// How the first-layer weight-gradient kernel cuts a set's positions: chunks of CW_CHUNK, slabs of at most
// WG_SAFE_LEN positions (at least two when a shard's sums must pass through the range check), blocks per plane.
ConvSmallWgradGeom conv_small_wgrad_plan(const ff_layer_desc& L, int B, int sm_count, bool two_slabs) {
  ConvSmallWgradGeom g;
  g.H = L.H, g.W = L.Wd, g.Ho = tc_out_h(L), g.Wo = tc_out_w(L), g.stride = tc_conv_stride(L), g.B = B;
  g.rows_per_pass = B * g.Ho * g.Wo;
  g.chunks = (g.rows_per_pass + CW_CHUNK - 1) / CW_CHUNK;
  const int safe_chunks = (int)(WG_SAFE_LEN / CW_CHUNK);
  g.n_slabs = (g.chunks + safe_chunks - 1) / safe_chunks;
  if (two_slabs && g.n_slabs < 2) g.n_slabs = 2;
  g.chunks_per_slab = (g.chunks + g.n_slabs - 1) / g.n_slabs;
  const int planes = 2 * g.n_slabs;
  g.blocks_per_plane = sm_count * 2 / planes;
  if (g.blocks_per_plane > g.chunks_per_slab) g.blocks_per_plane = g.chunks_per_slab;
  if (g.blocks_per_plane < 1) g.blocks_per_plane = 1;
  return g;
}

ff_status conv_small_wgrad(ff_ctx* ctx, const ff_layer_desc& L, const ff_layer_bufs& b, int B, cudaStream_t st) {
  const ConvSmallWgradGeom g = conv_small_wgrad_plan(L, B, ctx->sm_count, dp_checks_needed(ctx, L));
  const int planes = 2 * g.n_slabs;
  const size_t bytes = (size_t)planes * L.N * L.K * sizeof(int32_t);
  if (ctx->workspace_bytes < WS_BYTES + bytes) return fail(ctx, FF_ERR_WORKSPACE, "workspace has no room for the weight-gradient slabs");
  int32_t* slabs = reinterpret_cast<int32_t*>(static_cast<char*>(ctx->workspace) + WS_BYTES);
  ProfScope prof(ctx, FF_K_UPD_GEMM, st);
  const bool was = ctx->profiling;
  ctx->profiling = false;  // one event pair around the route
  if (cudaMemsetAsync(slabs, 0, bytes, st) != cudaSuccess) {
    ctx->profiling = was;
    return fail(ctx, FF_ERR_CUDA, "cudaMemsetAsync failed");
  }
  const int grid = planes * g.blocks_per_plane;
#define FF_CW_LAUNCH(CIN, NN) conv3x3_small_wgrad_kernel<CIN, NN><<<grid, CS_THREADS, 0, st>>>(b.Xq, b.dHq, slabs, g)
#define FF_CW_BY_N(CIN)                  \
  switch (L.N) {                         \
    case 16: FF_CW_LAUNCH(CIN, 16); break; \
    case 32: FF_CW_LAUNCH(CIN, 32); break; \
    case 64: FF_CW_LAUNCH(CIN, 64); break; \
    default: FF_CW_LAUNCH(CIN, 128); break; \
  }
  switch (L.Cin) {
    case 1: FF_CW_BY_N(1); break;
    case 2: FF_CW_BY_N(2); break;
    case 3: FF_CW_BY_N(3); break;
    default: FF_CW_BY_N(4); break;
  }
#undef FF_CW_BY_N
#undef FF_CW_LAUNCH
  ff_status s = FF_OK;
  if (cudaPeekAtLastError() != cudaSuccess) s = fail(ctx, FF_ERR_CUDA, "weight-gradient launch failed: %s", cudaGetErrorString(cudaGetLastError()));
  if (s == FF_OK) {
    ctx->launches++;
    s = launch_slab_update(ctx, slabs, g.n_slabs, L, b, st, 0);
  }
  ctx->profiling = was;
  return s;
}

ff_status run_forward_gemm(ff_ctx* ctx, const ff_layer_desc& L, const ff_layer_bufs& b, int B, cudaStream_t st) {
  if (L.kind == FF_DWCONV3X3) return dw_forward(ctx, L, b, B, st);
  if (ctx->gemm_path == FF_GEMM_AUTO && conv_small_ok(L.kind == FF_CONV3X3, L.Cin, L.N)) return conv_small_forward(ctx, L, b, B, st);
  const int R = rows_per_sample(L);
  const int rows = 2 * B * R;
  bool tc_ok = tc_forward_supported(L, B);
  if (!tc_ok && im2col_route(ctx, L, B)) {
    const Im2colPlan pl = im2col_plan(L, B, ctx->workspace_bytes, ctx->sm_count);
    ProfScope prof(ctx, FF_K_FWD_GEMM, st);
    const bool was = ctx->profiling;
    ctx->profiling = false;  // one event pair around the whole route
    ff_status s = launch_im2col(ctx, L, b, B, pl, true, st);
    ctx->profiling = was;
    if (s != FF_OK) return s;
    const char* ws = static_cast<const char*>(ctx->workspace);
    s = tc_forward(ctx->tc, L, b, B, status_ptr(ctx), st, reinterpret_cast<const int8_t*>(ws + pl.xi_off),
                   reinterpret_cast<const int8_t*>(ws + pl.wi_off), pl.kpad);
    if (s != FF_OK) return fail(ctx, s, "tensor-core forward launch failed: %s", ctx->tc.err);
    ctx->launches++;
    return FF_OK;
  }
  if (ctx->gemm_path == FF_GEMM_TENSOR && !tc_ok) return fail(ctx, FF_ERR_ARG, "shape not supported by the tensor-core forward");
  if (tc_ok && ctx->gemm_path != FF_GEMM_SIMT) {
    ProfScope prof(ctx, FF_K_FWD_GEMM, st);
    ff_status s = tc_forward(ctx->tc, L, b, B, status_ptr(ctx), st);
    if (s != FF_OK) return fail(ctx, s, "tensor-core forward launch failed: %s", ctx->tc.err);
    ctx->launches++;
    return FF_OK;
  }
  ForwardEpilogue epi{b.Y, b.acc_dump, reinterpret_cast<unsigned long long*>(b.S), b.rowmax, b.absmax, rows, L.N, B * R, R};
  if (L.kind != FF_CONV3X3)
    return launch_simt<DenseView, DenseView, false, 1>(ctx, dense(b.Xq, rows, L.K, b.ld_xq), dense(b.Wq, L.N, L.K), rows, L.N, L.K, epi, st);
  return launch_simt<Im2colView, DenseView, false, 1>(ctx, im2col(b.Xq, L, 2 * B), dense(b.Wq, L.N, L.K), rows, L.N, L.K, epi, st);
}

ff_status run_update_gemm(ff_ctx* ctx, const ff_layer_desc& L, const ff_layer_bufs& b, int B, cudaStream_t st);

inline size_t adam_plane_bytes(const ff_layer_desc& L) { return up256((size_t)2 * L.N * L.K * sizeof(int32_t)); }

// Adam layers: the weight-gradient routes only accumulate (INT32 sums of both sets into one dense plane: the
// caller's accW_dump if given, else the tail of the workspace, which the routes are kept out of meanwhile),
// then the common update kernel applies the rule.  The fused update epilogues stay as they are.
ff_status run_update_adam(ff_ctx* ctx, const ff_layer_desc& L, const ff_layer_bufs& b, int B, cudaStream_t st) {
  if (!b.Mom || !b.Var) return fail(ctx, FF_ERR_ARG, "the Adam update needs the buffers Mom and Var");
  if (ctx->accumulate_only) {  // data-parallel phase: sums go to accW_dump (checked by the caller), update comes later
    ff_layer_desc plain = L;
    plain.optimizer = FF_OPT_SGD;
    return run_update_gemm(ctx, plain, b, B, st);
  }
  ff_layer_bufs b2 = b;
  const size_t saved = ctx->workspace_bytes;
  if (!b2.accW_dump) {
    const size_t bytes = adam_plane_bytes(L);
    if (saved < WS_BYTES + bytes) return fail(ctx, FF_ERR_WORKSPACE, "workspace has no room for the Adam layer's weight-gradient sums");
    const size_t off = (saved - bytes) / 256 * 256;
    b2.accW_dump = reinterpret_cast<int32_t*>(static_cast<char*>(ctx->workspace) + off);
    ctx->workspace_bytes = off;
  }
  ff_layer_desc plain = L;
  plain.optimizer = FF_OPT_SGD;
  ctx->accumulate_only = true;
  ff_status s = run_update_gemm(ctx, plain, b2, B, st);
  ctx->accumulate_only = false;
  ctx->workspace_bytes = saved;
  if (s != FF_OK) return s;
  ProfScope prof(ctx, FF_K_UPD_GEMM, st);
  return launch_slab_update(ctx, b2.accW_dump, 1, L, b2, st);
}

// Weight-gradient contraction + fused update.
ff_status run_update_gemm(ff_ctx* ctx, const ff_layer_desc& L, const ff_layer_bufs& b, int B, cudaStream_t st) {
  if (L.optimizer == FF_OPT_ADAM) return run_update_adam(ctx, L, b, B, st);
  if (L.momentum != 0.0f && !b.Mom) return fail(ctx, FF_ERR_ARG, "momentum != 0 needs the buffer Mom");
  if (L.kind == FF_DWCONV3X3) return dw_update(ctx, L, b, B, st);
  const int R = rows_per_sample(L);
  const int rows = 2 * B * R;
  if (ctx->gemm_path == FF_GEMM_AUTO && conv_small_ok(L.kind == FF_CONV3X3, L.Cin, L.N)) return conv_small_wgrad(ctx, L, b, B, st);
  bool tc_ok = tc_update_supported(L, B);
  if (!tc_ok && L.N % 16 == 0 && im2col_route(ctx, L, B)) {
    // explicit im2col (rebuilt from Xq: the workspace is transient), dense split contraction into slabs, reduce + update
    const Im2colPlan pl = im2col_plan(L, B, ctx->workspace_bytes, ctx->sm_count);
    ProfScope prof(ctx, FF_K_UPD_GEMM, st);
    const bool was = ctx->profiling;
    ctx->profiling = false;
    ff_status s = launch_im2col(ctx, L, b, B, pl, false, st);
    if (s == FF_OK) {
      char* ws = static_cast<char*>(ctx->workspace);
      int32_t* slabs = reinterpret_cast<int32_t*>(ws + pl.slab_off);
      int used = 0;
      s = tc_dense_update_slab(ctx->tc, b.dHq, L.N, reinterpret_cast<const int8_t*>(ws + pl.xi_off), pl.kpad, B * R, slabs,
                               pl.max_splits, &used, status_ptr(ctx), st);
      if (s != FF_OK) {
        ctx->profiling = was;
        return fail(ctx, s, "tensor-core weight-gradient launch failed: %s", ctx->tc.err);
      }
      ctx->launches++;
      s = launch_slab_update(ctx, slabs, used, L, b, st, pl.kpad);
    }
    ctx->profiling = was;
    return s;
  }
  if (ctx->gemm_path == FF_GEMM_TENSOR && !tc_ok) return fail(ctx, FF_ERR_ARG, "shape not supported by the tensor-core weight gradient");
  if (tc_ok && ctx->gemm_path != FF_GEMM_SIMT && L.kind == FF_CONV1X1) {
    // pointwise convolution: a dense contraction over every position of a set.  With few output tiles it is
    // split into INT32 slabs like the 3x3 case; otherwise the fused dense kernel below takes it.
    int splits = tc_dense_slab_splits(L.N, L.K, (long long)B * R, ctx->sm_count);
    int need = tc_min_splits(((long long)B * R + 127) / 128);
    if (dp_checks_needed(ctx, L) && need < 2) need = 2;
    if (splits < need) splits = need;
    const size_t room = ctx->workspace_bytes > WS_BYTES ? ctx->workspace_bytes - WS_BYTES : 0;
    const size_t per_split = (size_t)2 * L.N * L.K * sizeof(int32_t);
    if ((size_t)splits * per_split > room) splits = (int)(room / per_split);
    if (splits < need) return fail(ctx, FF_ERR_WORKSPACE, "workspace has no room for the weight-gradient slabs");
    if (splits >= 2) {
      int32_t* slabs = reinterpret_cast<int32_t*>(static_cast<char*>(ctx->workspace) + WS_BYTES);
      ProfScope prof(ctx, FF_K_UPD_GEMM, st);
      int used = 0;
      ff_status s = tc_dense_update_slab(ctx->tc, b.dHq, L.N, b.Xq, L.K, B * R, slabs, splits, &used, status_ptr(ctx), st,
                                         b.ld_dhq, b.ld_xq);
      if (s != FF_OK) return fail(ctx, s, "tensor-core weight-gradient launch failed: %s", ctx->tc.err);
      ctx->launches++;
      const bool was = ctx->profiling;
      ctx->profiling = false;
      s = launch_slab_update(ctx, slabs, used, L, b, st);
      ctx->profiling = was;
      return s;
    }
  }
  if (tc_ok && ctx->gemm_path != FF_GEMM_SIMT && L.kind != FF_CONV3X3) {
    ProfScope prof(ctx, FF_K_UPD_GEMM, st);
    int used = 0;
    // accumulate only: one unsplit contraction whose single slab [2][N][K] is accW_dump itself
    ff_status s = ctx->accumulate_only ? tc_dense_update_slab(ctx->tc, b.dHq, L.N, b.Xq, L.K, B * R, b.accW_dump, 1, &used,
                                                              status_ptr(ctx), st, b.ld_dhq, b.ld_xq)
                                       : tc_update(ctx->tc, L, b, B * R, status_ptr(ctx), st);
    if (s != FF_OK) return fail(ctx, s, "tensor-core weight-gradient launch failed: %s", ctx->tc.err);
    ctx->launches++;
    return FF_OK;
  }
  if (tc_ok && ctx->gemm_path != FF_GEMM_SIMT) {
    // convolution: split implicit-GEMM contraction into INT32 slabs in the workspace, then reduce + update
    int splits = tc_conv_update_splits(L, B, ctx->sm_count, ctx->tc.force_ncta);
    const size_t room = ctx->workspace_bytes > WS_BYTES ? ctx->workspace_bytes - WS_BYTES : 0;
    const size_t per_split = tc_conv_update_slab_bytes(L, 1);
    if ((size_t)splits * per_split > room) splits = (int)(room / per_split);
    if (splits >= tc_min_splits((long long)B * R / 128)) {
      int32_t* slabs = reinterpret_cast<int32_t*>(static_cast<char*>(ctx->workspace) + WS_BYTES);
      ProfScope prof(ctx, FF_K_UPD_GEMM, st);
      int used = 0;
      ff_status s = tc_conv_update(ctx->tc, L, b, B, slabs, splits, &used, status_ptr(ctx), st);
      if (s != FF_OK) return fail(ctx, s, "tensor-core convolution weight-gradient launch failed: %s", ctx->tc.err);
      ctx->launches++;
      const bool was = ctx->profiling;
      ctx->profiling = false;
      s = launch_slab_update(ctx, slabs, used, L, b, st);
      ctx->profiling = was;
      return s;
    }
    if (ctx->gemm_path == FF_GEMM_TENSOR) return fail(ctx, FF_ERR_WORKSPACE, "workspace has no room for the weight-gradient slabs");
  }
  const int clen = B * R;
  int splits = simt_wgrad_splits(L, B, ctx->workspace_bytes);
  if (splits < simt_min_splits(L, B)) return fail(ctx, FF_ERR_WORKSPACE, "workspace has no room for the weight-gradient slabs");
  if (dp_checks_needed(ctx, L) && splits < 2) {
    if (ctx->workspace_bytes < WS_BYTES + (size_t)4 * L.N * L.K * sizeof(int32_t))
      return fail(ctx, FF_ERR_WORKSPACE, "workspace has no room for the weight-gradient slabs");
    splits = 2;
  }
  if (splits > 1) {
    // few output tiles, long contraction: split it, keep INT32 partial sums in the workspace, add them exactly
    int32_t* slabs = reinterpret_cast<int32_t*>(static_cast<char*>(ctx->workspace) + WS_BYTES);
    SlabEpilogue epi{slabs, L.N, L.K};
    ff_status s;
    {
      ProfScope prof(ctx, FF_K_UPD_GEMM, st);
      const bool was = ctx->profiling;
      ctx->profiling = false;  // one event pair around both launches
      if (L.kind != FF_CONV3X3)
        s = launch_simt<DenseView, DenseView, true, 2>(ctx, dense(b.dHq, rows, L.N, b.ld_dhq), dense(b.Xq, rows, L.K, b.ld_xq), L.N, L.K, clen, epi, st, splits);
      else
        s = launch_simt<DenseView, Im2colView, true, 2>(ctx, dense(b.dHq, rows, L.N), im2col(b.Xq, L, 2 * B), L.N, L.K, clen, epi, st, splits);
      if (s == FF_OK) s = launch_slab_update(ctx, slabs, simt_split_count(clen, splits), L, b, st);
      ctx->profiling = was;
    }
    return s;
  }
  if (ctx->accumulate_only) {
    SlabEpilogue epi{b.accW_dump, L.N, L.K};
    if (L.kind != FF_CONV3X3)
      return launch_simt<DenseView, DenseView, true, 2>(ctx, dense(b.dHq, rows, L.N, b.ld_dhq), dense(b.Xq, rows, L.K, b.ld_xq), L.N, L.K, clen, epi, st);
    return launch_simt<DenseView, Im2colView, true, 2>(ctx, dense(b.dHq, rows, L.N), im2col(b.Xq, L, 2 * B), L.N, L.K, clen, epi, st);
  }
  UpdateEpilogue epi{b.W, b.accW_dump, b.absmax, L.lr, L.N, L.K, L.momentum != 0.0f ? b.Mom : nullptr, L.momentum};
  if (L.kind != FF_CONV3X3)
    return launch_simt<DenseView, DenseView, true, 2>(ctx, dense(b.dHq, rows, L.N, b.ld_dhq), dense(b.Xq, rows, L.K, b.ld_xq), L.N, L.K, clen, epi, st);
  return launch_simt<DenseView, Im2colView, true, 2>(ctx, dense(b.dHq, rows, L.N), im2col(b.Xq, L, 2 * B), L.N, L.K, clen, epi, st);
}

// ---- step pieces --------------------------------------------------------------------------
// Quantise the weights and run the forward contraction; the layer input is already in Xq and
// its ranges in absmax[X_POS..X_NEG].
ff_status forward_from_xq(ff_ctx* ctx, const ff_layer_desc& L, const ff_layer_bufs& b, int B,
                          float* a_next2, cudaStream_t st, bool weights_ready = false) {
  const size_t nW = (size_t)L.N * L.K;
  if (!weights_ready) {
    ProfScope prof(ctx, FF_K_ABSMAX, st);
    absmax_kernel<<<dim3(ew_blocks(ctx, nW / 4 + 1), 1), EW_THREADS, 0, st>>>(b.W, nW, b.absmax + FF_A_W, status_ptr(ctx));
  }
  if (!weights_ready) FF_LAUNCH_CHECK(ctx);
  if (!weights_ready) {
    ProfScope prof(ctx, FF_K_QUANTIZE, st);
    const dim3 grid(ew_blocks(ctx, nW / 4 + 1), 1);
    const KeySpec key = make_key_spec(L.seed, ROLE_W, L.index, step_ptr(ctx));
    unsigned long long* S = reinterpret_cast<unsigned long long*>(b.S);  // cleared on the side for the forward epilogue
    if (L.round_w == FF_ROUND_NEAREST_EVEN)
      quantize_kernel<ROUND_NEAREST><<<grid, EW_THREADS, 0, st>>>(b.W, b.Wq, nW, b.absmax + FF_A_W, key, S, b.rowmax, 2 * B);
    else
      quantize_kernel<ROUND_STOCHASTIC><<<grid, EW_THREADS, 0, st>>>(b.W, b.Wq, nW, b.absmax + FF_A_W, key, S, b.rowmax, 2 * B);
  }
  if (!weights_ready) FF_LAUNCH_CHECK(ctx);
  ff_status s = run_forward_gemm(ctx, L, b, B, st);
  if (s != FF_OK) return s;
  {
    ProfScope prof(ctx, FF_K_FINALIZE, st);
    finalize_goodness_kernel<<<dim3(ew_blocks(ctx, B, 1), 2), EW_THREADS, 0, st>>>(
        reinterpret_cast<const unsigned long long*>(b.S), b.rowmax, b.absmax, B, L.tau, L.eps, b.G,
        b.absmax + FF_A_XNEXT_POS, a_next2, b.Skip ? 0 : (ctx->joint_range ? 2 : 1), factors_ptr(ctx, B));
  }
  FF_LAUNCH_CHECK(ctx);
  return FF_OK;
}

ff_status quantize_input(ff_ctx* ctx, const ff_layer_desc& L, const ff_layer_bufs& b, int B, cudaStream_t st,
                         bool do_absmax = true, bool do_quantize = true) {
  const size_t per_sample = (size_t)in_rows_per_sample(L) * in_features(L);
  const size_t per_pass = (size_t)B * per_sample;
  if (do_absmax) {
    ProfScope prof(ctx, FF_K_ABSMAX, st);
    absmax_kernel<<<dim3(ew_blocks(ctx, per_pass / 4 + 1), 2), EW_THREADS, 0, st>>>(b.X, per_pass, b.absmax + FF_A_X_POS,
                                                                                 status_ptr(ctx), ctx->joint_range ? 1 : 0);
  }
  if (do_absmax) FF_LAUNCH_CHECK(ctx);
  if (!do_quantize) return FF_OK;
  {
    ProfScope prof(ctx, FF_K_QUANTIZE, st);
    const dim3 grid(ew_blocks(ctx, per_pass / 4 + 1), 2);
    const KeySpec key = make_key_spec(L.seed, ROLE_X, L.index, step_ptr(ctx));
    const uint2 bias = ctr_bias(ctx, per_sample, B);
    if (L.round_x == FF_ROUND_NEAREST_EVEN)
      quantize_kernel<ROUND_NEAREST><<<grid, EW_THREADS, 0, st>>>(b.X, b.Xq, per_pass, b.absmax + FF_A_X_POS, key, nullptr,
                                                                 nullptr, 0, bias, row_pad(L.K, b.ld_xq));
    else
      quantize_kernel<ROUND_STOCHASTIC><<<grid, EW_THREADS, 0, st>>>(b.X, b.Xq, per_pass, b.absmax + FF_A_X_POS, key, nullptr,
                                                                    nullptr, 0, bias, row_pad(L.K, b.ld_xq));
  }
  FF_LAUNCH_CHECK(ctx);
  return FF_OK;
}

// Normalised output of layer `L` as FP32 (b.Xnext, if non-NULL) and / or as the INT8 input of the
// next layer (xq_next, nullable; rounding keyed by the next layer).
ff_status normalize_output(ff_ctx* ctx, const ff_layer_desc& L, const ff_layer_bufs& b, int B, int8_t* xq_next,
                           const ff_layer_desc* next, cudaStream_t st, int ld_next = 0, float* a_next2 = nullptr) {
  if (!b.Xnext && !xq_next) return FF_OK;
  if (b.Skip) {
    // residual block: the sum of the normalised output and the skip tensor goes to Xnext in FP32 together with its
    // range (it has no short-cut), then the ordinary quantiser makes the next layer's INT8 input from it
    if (ctx->shard.B_total) return fail(ctx, FF_ERR_ARG, "a data-parallel step takes no skip paths");
    const size_t per_sample = (size_t)rows_per_sample(L) * L.N, per_pass = per_sample * B;
    const dim3 grid(ew_blocks(ctx, per_pass / 4 + 1), 2);
    {
      ProfScope prof(ctx, FF_K_NORMALIZE, st);
      normalize_skip_kernel<<<grid, EW_THREADS, 0, st>>>(b.Y, b.G, L.tau, L.eps, per_sample, per_pass, b.Skip, L.skip_scale, b.Xnext,
                                                        b.absmax + FF_A_XNEXT_POS, a_next2, status_ptr(ctx),
                                                        ctx->joint_range ? 1 : 0);
    }
    FF_LAUNCH_CHECK(ctx);
    if (!xq_next) return FF_OK;
    ProfScope prof(ctx, FF_K_QUANTIZE, st);
    const KeySpec key = make_key_spec(next->seed, ROLE_X, next->index, step_ptr(ctx));
    const RowPad rp = row_pad((int)per_sample, ld_next);
    if (next->round_x == FF_ROUND_NEAREST_EVEN)
      quantize_kernel<ROUND_NEAREST><<<grid, EW_THREADS, 0, st>>>(b.Xnext, xq_next, per_pass, b.absmax + FF_A_XNEXT_POS, key, nullptr,
                                                                 nullptr, 0, uint2{0u, 0u}, rp);
    else
      quantize_kernel<ROUND_STOCHASTIC><<<grid, EW_THREADS, 0, st>>>(b.Xnext, xq_next, per_pass, b.absmax + FF_A_XNEXT_POS, key, nullptr,
                                                                    nullptr, 0, uint2{0u, 0u}, rp);
    FF_LAUNCH_CHECK(ctx);
    return FF_OK;
  }
  if (ld_next && L.pool == 2) return fail(ctx, FF_ERR_ARG, "a pooled output cannot feed a layer with a padded Xq");
  const size_t per_sample = (size_t)rows_per_sample(L) * L.N;
  const size_t per_pass = per_sample * B;
  const KeySpec key = next ? make_key_spec(next->seed, ROLE_X, next->index, step_ptr(ctx)) : KeySpec{0ull, step_ptr(ctx)};
  if (L.pool == 2) {
    ProfScope prof(ctx, FF_K_NORMALIZE, st);
    const bool stoch = next && next->round_x != FF_ROUND_NEAREST_EVEN;
    const bool vec = L.N % 4 == 0;
    const int Ho = tc_out_h(L), Wo = tc_out_w(L);
    const dim3 grid(ew_blocks(ctx, per_pass / 4 / (vec ? 4 : 1) + 1, 1), 2);
    const uint2 bias = ctr_bias(ctx, per_sample / 4, B);
    const float* a = b.absmax + FF_A_XNEXT_POS;
    if (vec && stoch)
      normalize_pool_kernel<ROUND_STOCHASTIC, 4><<<grid, EW_THREADS, 0, st>>>(b.Y, b.G, L.tau, L.eps, B, Ho, Wo, L.N, b.Xnext,
                                                                             xq_next, a, key, bias);
    else if (vec)
      normalize_pool_kernel<ROUND_NEAREST, 4><<<grid, EW_THREADS, 0, st>>>(b.Y, b.G, L.tau, L.eps, B, Ho, Wo, L.N, b.Xnext, xq_next,
                                                                          a, key, bias);
    else if (stoch)
      normalize_pool_kernel<ROUND_STOCHASTIC, 1><<<grid, EW_THREADS, 0, st>>>(b.Y, b.G, L.tau, L.eps, B, Ho, Wo, L.N, b.Xnext,
                                                                             xq_next, a, key, bias);
    else
      normalize_pool_kernel<ROUND_NEAREST, 1><<<grid, EW_THREADS, 0, st>>>(b.Y, b.G, L.tau, L.eps, B, Ho, Wo, L.N, b.Xnext, xq_next,
                                                                          a, key, bias);
    FF_LAUNCH_CHECK(ctx);
    return FF_OK;
  }
  {
    ProfScope prof(ctx, FF_K_NORMALIZE, st);
    const dim3 grid(ew_blocks(ctx, per_pass / 4 + 1), 2);
    const uint2 bias = ctr_bias(ctx, per_sample, B);
    const bool nearest = !next || next->round_x == FF_ROUND_NEAREST_EVEN;
    const RowPad rp = row_pad((int)per_sample, ld_next);
    const float* a = b.absmax + FF_A_XNEXT_POS;
    if (nearest && !rp.extra)
      normalize_kernel<ROUND_NEAREST, false><<<grid, EW_THREADS, 0, st>>>(b.Y, b.G, L.tau, L.eps, per_sample, per_pass, b.Xnext,
                                                                         xq_next, a, key, bias, RowPad{0u, 0u}, factors_ptr(ctx, B));
    else if (nearest)
      normalize_kernel<ROUND_NEAREST, true><<<grid, EW_THREADS, 0, st>>>(b.Y, b.G, L.tau, L.eps, per_sample, per_pass, b.Xnext,
                                                                        xq_next, a, key, bias, rp, factors_ptr(ctx, B));
    else if (!rp.extra)
      normalize_kernel<ROUND_STOCHASTIC, false><<<grid, EW_THREADS, 0, st>>>(b.Y, b.G, L.tau, L.eps, per_sample, per_pass, b.Xnext,
                                                                            xq_next, a, key, bias, RowPad{0u, 0u}, factors_ptr(ctx, B));
    else
      normalize_kernel<ROUND_STOCHASTIC, true><<<grid, EW_THREADS, 0, st>>>(b.Y, b.G, L.tau, L.eps, per_sample, per_pass, b.Xnext,
                                                                           xq_next, a, key, bias, rp, factors_ptr(ctx, B));
  }
  FF_LAUNCH_CHECK(ctx);
  return FF_OK;
}

ff_status loss_grad_impl(ff_ctx* ctx, const ff_layer_desc& L, const ff_layer_bufs& b, int B, const float* const* G_later,
                         const float* theta_later, int n_later, float lambda, cudaStream_t st, bool do_loss = true,
                         bool do_dh = true) {
  LaterLayers later;
  later.n = n_later;
  for (int j = 0; j < n_later; ++j) {
    later.G[j] = G_later[j];
    later.theta[j] = theta_later[j];
  }
  int loss_blocks = (2 * B + LOSS_THREADS - 1) / LOSS_THREADS;
  if (loss_blocks > LOSS_MAX_BLOCKS) loss_blocks = LOSS_MAX_BLOCKS;
  if (do_loss) {
    ProfScope prof(ctx, FF_K_LOSS, st);
    loss_coef_kernel<<<loss_blocks, LOSS_THREADS, 0, st>>>(
        b.G, L.theta, later, lambda, B, b.rowmax, b.absmax, b.coef, b.loss,
        reinterpret_cast<LossScratch*>(static_cast<char*>(ctx->workspace) + WS_LOSS_OFFSET), step_ptr(ctx),
        2 * ctx->shard.B_total);
  }
  if (do_loss) FF_LAUNCH_CHECK(ctx);
  if (!do_dh) return FF_OK;
  const size_t per_sample = (size_t)rows_per_sample(L) * L.N;
  const size_t per_pass = per_sample * B;
  {
    ProfScope prof(ctx, FF_K_DH_QUANTIZE, st);
    const dim3 grid(ew_blocks(ctx, per_pass / 4 + 1), 2);
    const KeySpec key = make_key_spec(L.seed, ROLE_DH, L.index, step_ptr(ctx));
    const uint2 bias = ctr_bias(ctx, per_sample, B);
    if (L.round_dh == FF_ROUND_NEAREST_EVEN)
      dh_quantize_kernel<ROUND_NEAREST><<<grid, EW_THREADS, 0, st>>>(b.Y, b.coef, b.absmax, per_sample, per_pass, b.dHq, key, bias,
                                                                    row_pad(L.N, b.ld_dhq));
    else
      dh_quantize_kernel<ROUND_STOCHASTIC><<<grid, EW_THREADS, 0, st>>>(b.Y, b.coef, b.absmax, per_sample, per_pass, b.dHq, key,
                                                                       bias, row_pad(L.N, b.ld_dhq));
  }
  FF_LAUNCH_CHECK(ctx);
  return FF_OK;
}

ff_status check_layer_list(ff_ctx* ctx, const ff_layer_desc* layers, const ff_layer_bufs* bufs, int n_layers, int B) {
  if (!layers || !bufs || n_layers <= 0 || n_layers > FF_MAX_LATER + 1) return fail(ctx, FF_ERR_ARG, "bad layer list");
  ff_status s;
  for (int l = 0; l < n_layers; ++l) {
    if ((s = check_layer(ctx, &layers[l], B)) != FF_OK) return s;
    if ((s = check_bufs(ctx, &bufs[l], l == 0)) != FF_OK) return s;
    if ((s = check_pitches(ctx, &layers[l], &bufs[l])) != FF_OK) return s;
    if (l > 0 && !bufs[l].X) {
      const ff_layer_desc &p = layers[l - 1], &c = layers[l];
      if (next_values_per_sample(p) != (long long)in_rows_per_sample(c) * in_features(c))
        return fail(ctx, FF_ERR_ARG, "layer output / next layer input sizes differ");
    }
  }
  return FF_OK;
}

// INT8 forward through all layers with the current weights (Alg. 1, forward pass): layer 0 reads bufs[0].X,
// layer l > 0 reads bufs[l].X if given, else the previous layer's normalised output, quantised on the fly.
// Everything a step can quantise before any layer has run, in two launches whatever the number of layers:
// ranges of the network input (both sets) and of every layer's weights, then their INT8 codes (which also
// clears the forward epilogues' per-sample accumulators).  The range vectors were cleared by set_step.
ff_status quantize_inputs_and_weights(ff_ctx* ctx, const ff_layer_desc* layers, const ff_layer_bufs* bufs, int n, int B,
                                      cudaStream_t st) {
  AbsmaxJobs aj;
  QuantJobs qj;
  int t = 0;
  size_t largest = 0;
  const ff_layer_desc& L0 = layers[0];
  const size_t per_sample0 = (size_t)in_rows_per_sample(L0) * in_features(L0), per_pass0 = per_sample0 * B;
  const uint2 bias0 = ctr_bias(ctx, per_sample0, B);
  for (int p = 0; p < 2; ++p, ++t) {
    aj.x[t] = bufs[0].X + p * per_pass0, aj.n[t] = per_pass0, aj.out[t] = bufs[0].absmax + FF_A_X_POS + p;
    aj.out2[t] = ctx->joint_range ? bufs[0].absmax + FF_A_X_POS + (p ^ 1) : nullptr;
    qj.x[t] = aj.x[t], qj.q[t] = bufs[0].Xq, qj.e0[t] = p * per_pass0, qj.n[t] = per_pass0, qj.a[t] = aj.out[t];
    qj.pad[t] = row_pad(L0.K, bufs[0].ld_xq);
    qj.s1[t] = make_key_spec(L0.seed, ROLE_X, L0.index, nullptr).s1;
    qj.ctr0[t] = (uint32_t)(p * per_pass0) + (p ? bias0.y : bias0.x);
    qj.stochastic[t] = L0.round_x != FF_ROUND_NEAREST_EVEN;
  }
  largest = per_pass0;
  for (int l = 0; l < n; ++l, ++t) {
    const size_t nW = (size_t)layers[l].N * layers[l].K;
    aj.x[t] = bufs[l].W, aj.n[t] = nW, aj.out[t] = bufs[l].absmax + FF_A_W, aj.out2[t] = nullptr;
    qj.x[t] = bufs[l].W, qj.q[t] = bufs[l].Wq, qj.n[t] = nW, qj.a[t] = aj.out[t];
    qj.s1[t] = make_key_spec(layers[l].seed, ROLE_W, layers[l].index, nullptr).s1;
    qj.ctr0[t] = 0u;
    qj.e0[t] = 0, qj.pad[t] = RowPad{0u, 0u};
    qj.stochastic[t] = layers[l].round_w != FF_ROUND_NEAREST_EVEN;
    qj.zero_S[l] = reinterpret_cast<unsigned long long*>(bufs[l].S);
    qj.zero_rowmax[l] = bufs[l].rowmax;
    if (nW > largest) largest = nW;
  }
  qj.n_zero = n, qj.zero_n = 2 * B, qj.ss = step_ptr(ctx);
  const dim3 grid(ew_blocks(ctx, largest / 4 + 1), t);
  {
    ProfScope prof(ctx, FF_K_ABSMAX, st);
    absmax_multi_kernel<<<grid, EW_THREADS, 0, st>>>(aj, status_ptr(ctx));
  }
  FF_LAUNCH_CHECK(ctx);
  {
    ProfScope prof(ctx, FF_K_QUANTIZE, st);
    if (bufs[0].ld_xq)
      quantize_multi_kernel<true><<<grid, EW_THREADS, 0, st>>>(qj);
    else
      quantize_multi_kernel<false><<<grid, EW_THREADS, 0, st>>>(qj);
  }
  FF_LAUNCH_CHECK(ctx);
  return FF_OK;
}

ff_status forward_all(ff_ctx* ctx, const ff_layer_desc* layers, const ff_layer_bufs* bufs, int n_layers, int B,
                      cudaStream_t st) {
  ff_status s;
  if ((s = quantize_inputs_and_weights(ctx, layers, bufs, n_layers, B, st)) != FF_OK) return s;
  for (int l = 0; l < n_layers; ++l) {
    const bool chained = l > 0 && !bufs[l].X;
    if (l > 0 && !chained && (s = quantize_input(ctx, layers[l], bufs[l], B, st)) != FF_OK) return s;
    const bool feeds_next = l + 1 < n_layers && !bufs[l + 1].X;
    if ((s = forward_from_xq(ctx, layers[l], bufs[l], B, feeds_next ? bufs[l + 1].absmax + FF_A_X_POS : nullptr, st, true)) != FF_OK)
      return s;
    if ((s = normalize_output(ctx, layers[l], bufs[l], B, feeds_next ? bufs[l + 1].Xq : nullptr,
                              feeds_next ? &layers[l + 1] : nullptr, st, feeds_next ? bufs[l + 1].ld_xq : 0,
                              feeds_next ? bufs[l + 1].absmax + FF_A_X_POS : nullptr)) != FF_OK)
      return s;
  }
  return FF_OK;
}

// Everything of one train step after the step counter and lambda have been published (Alg. 1, epoch body).
// Layers before `first` are frozen: they take part in the forward only (layer-by-layer training, Sec. III).
ff_status train_step_body(ff_ctx* ctx, const ff_layer_desc* layers, const ff_layer_bufs* bufs, int n_layers, int B,
                          float lambda, cudaStream_t st, int first = 0) {
  ff_status s;
  (void)lambda;  // read by the kernels from the step state
  // Alg. 1, forward pass: one forward through all layers with the pre-update weights
  if ((s = forward_all(ctx, layers, bufs, n_layers, B, st)) != FF_OK) return s;
  // Alg. 1, per-layer loss and update: loss from the G's (Eq. 3) and INT8 output gradient - neither depends on an update, so all
  // layers share one launch each - then per layer the weight gradient and update
  LossJobs lj;
  DhJobs dj;
  lj.n = n_layers;
  size_t largest = 0;
  for (int l = 0; l < n_layers; ++l) {
    lj.G[l] = bufs[l].G, lj.theta[l] = layers[l].theta, lj.rowmax[l] = bufs[l].rowmax, lj.absmax[l] = bufs[l].absmax;
    lj.coef[l] = bufs[l].coef, lj.loss[l] = bufs[l].loss;
    dj.Y[l] = bufs[l].Y, dj.coef[l] = bufs[l].coef, dj.absmax[l] = bufs[l].absmax, dj.dHq[l] = bufs[l].dHq;
    dj.per_sample[l] = (unsigned long long)rows_per_sample(layers[l]) * layers[l].N;
    dj.s1[l] = make_key_spec(layers[l].seed, ROLE_DH, layers[l].index, nullptr).s1;
    dj.stochastic[l] = layers[l].round_dh != FF_ROUND_NEAREST_EVEN;
    dj.pad[l] = row_pad(layers[l].N, bufs[l].ld_dhq);
    if (l >= first && dj.per_sample[l] * B > largest) largest = dj.per_sample[l] * B;
  }
  dj.ss = step_ptr(ctx);
  int loss_blocks = (2 * B + LOSS_THREADS - 1) / LOSS_THREADS;
  if (loss_blocks > LOSS_MAX_BLOCKS) loss_blocks = LOSS_MAX_BLOCKS;
  {
    ProfScope prof(ctx, FF_K_LOSS, st);
    loss_coef_multi_kernel<<<dim3(loss_blocks, n_layers - first), LOSS_THREADS, 0, st>>>(
        lj, B, reinterpret_cast<LossScratch*>(static_cast<char*>(ctx->workspace) + WS_LOSS_OFFSET), step_ptr(ctx), 0, first);
  }
  FF_LAUNCH_CHECK(ctx);
  {
    ProfScope prof(ctx, FF_K_DH_QUANTIZE, st);
    bool any_pad = false;
    for (int l = first; l < n_layers; ++l) any_pad = any_pad || bufs[l].ld_dhq != 0;
    const dim3 grid(ew_blocks(ctx, largest / 4 + 1), 2 * (n_layers - first));
    if (any_pad)
      dh_quantize_multi_kernel<true><<<grid, EW_THREADS, 0, st>>>(dj, B, first);
    else
      dh_quantize_multi_kernel<false><<<grid, EW_THREADS, 0, st>>>(dj, B, first);
  }
  FF_LAUNCH_CHECK(ctx);
  for (int l = first; l < n_layers; ++l)
    if ((s = run_update_gemm(ctx, layers[l], bufs[l], B, st)) != FF_OK) return s;
  return FF_OK;
}

// One phase of the data-parallel step (see ff_dp_train_phase); ctx->shard is set by the caller.
ff_status dp_phase_body(ff_ctx* ctx, const ff_layer_desc* layers, const ff_layer_bufs* bufs, int n, int B, int phase,
                        float lambda, cudaStream_t st, ff_dp_reduce* red, int* n_red) {
  ff_status s;
  int nr = 0;
  // needed_by: the first phase that reads the combined array (the reduction may run beside the phases before it)
  auto want = [&](void* p, uint64_t count, int dtype, int op, int needed_by) {
    red[nr].dev_ptr = p;
    red[nr].count = count;
    red[nr].dtype = dtype;
    red[nr].op = op;
    red[nr].needed_by_phase = needed_by;
    ++nr;
  };
  if (phase == 0) {
    // ranges of the network input: local maxima now, the maximum over the shards before phase 1
    for (int l = 0; l < n; ++l) FF_CUDA(ctx, cudaMemsetAsync(bufs[l].absmax, 0, FF_ABSMAX_LEN * sizeof(float), st));
    if ((s = quantize_input(ctx, layers[0], bufs[0], B, st, true, false)) != FF_OK) return s;
    want(bufs[0].absmax + FF_A_X_POS, 2, FF_DP_F32, FF_DP_MAX, 1);
  } else if (phase <= n) {
    // forward of layer l; its input range is global by now, the range of its normalised output becomes so after the phase
    const int l = phase - 1;
    if (l == 0)
      s = quantize_input(ctx, layers[0], bufs[0], B, st, false, true);
    else
      s = normalize_output(ctx, layers[l - 1], bufs[l - 1], B, bufs[l].Xq, &layers[l], st, bufs[l].ld_xq);
    if (s != FF_OK) return s;
    const bool feeds_next = l + 1 < n;
    if ((s = forward_from_xq(ctx, layers[l], bufs[l], B, feeds_next ? bufs[l + 1].absmax + FF_A_X_POS : nullptr, st)) != FF_OK)
      return s;
    want(bufs[l].absmax + FF_A_XNEXT_POS, 2, FF_DP_F32, FF_DP_MAX, phase + 1);
    if (feeds_next) want(bufs[l + 1].absmax + FF_A_X_POS, 2, FF_DP_F32, FF_DP_MAX, phase + 1);
  } else if (phase == n + 1) {
    // FP32 output of the last layer (if asked for); losses and coefficients of all layers from the local G's
    if ((s = normalize_output(ctx, layers[n - 1], bufs[n - 1], B, nullptr, nullptr, st)) != FF_OK) return s;
    for (int l = 0; l < n; ++l) {
      const float* Gl[FF_MAX_LATER];
      float th[FF_MAX_LATER];
      const int n_later = n - 1 - l;
      for (int j = 0; j < n_later; ++j) {
        Gl[j] = bufs[l + 1 + j].G;
        th[j] = layers[l + 1 + j].theta;
      }
      if ((s = loss_grad_impl(ctx, layers[l], bufs[l], B, Gl, th, n_later, lambda, st, true, false)) != FF_OK) return s;
      want(bufs[l].absmax + FF_A_DH_POS, 2, FF_DP_F32, FF_DP_MAX, n + 2);   // range of dH over the whole batch
      want(bufs[l].loss, 1, FF_DP_F32, FF_DP_SUM, n + 2);                   // each shard holds its share of the batch mean
    }
  } else if (phase < 2 * n + 2) {
    // INT8 output gradient and the local INT32 weight-gradient sums of layer l.  Nothing reads the combined sums
    // before the layer's own update phase, so their (large) reduction can run beside the later layers' contractions.
    const int l = phase - (n + 2);
    ctx->accumulate_only = true;
    s = loss_grad_impl(ctx, layers[l], bufs[l], B, nullptr, nullptr, 0, lambda, st, false, true);
    if (s == FF_OK) s = run_update_gemm(ctx, layers[l], bufs[l], B, st);
    ctx->accumulate_only = false;
    if (s != FF_OK) return s;
    want(bufs[l].accW_dump, (uint64_t)2 * layers[l].N * layers[l].K, FF_DP_I32, FF_DP_SUM, 2 * n + 2 + l);
  } else {
    // the sums are those of the whole batch now: the same update on every device keeps the weights identical
    const int l = phase - (2 * n + 2);
    ProfScope prof(ctx, FF_K_UPD_GEMM, st);
    if ((s = launch_slab_update(ctx, bufs[l].accW_dump, 1, layers[l], bufs[l], st)) != FF_OK) return s;
  }
  *n_red = nr;
  return FF_OK;
}

constexpr size_t FF_MAX_GRAPHS = 16;

void drop_graphs(ff_ctx* ctx) {
  for (auto& g : ctx->graphs)
    if (g.exec) cudaGraphExecDestroy(g.exec);
  ctx->graphs.clear();
}

// Notes why a call shape stays on the eager path; readable through ff_last_error, no call fails because of it.
void graph_gave_up(ff_ctx* ctx, ff_ctx::GraphEntry* ent, const char* what, cudaError_t e) {
  ent->eager_only = true;
  snprintf(ctx->err, sizeof(ctx->err), "graph mode: %s (%s); this call shape runs kernel by kernel", what,
           cudaGetErrorString(e));
  cudaGetLastError();
}

// Train step through a captured launch sequence.  The sequence of a step depends on the layer list, the
// buffer pointers, the batch size, the workspace and the contraction route, but not on the step counter
// or lambda (those are read from device memory), so one captured graph serves every later step of the
// same call shape.  First call of a shape: eager (it also fills the per-kernel attribute and occupancy
// caches, which must not happen inside a capture).  Second call: captured, instantiated and launched.
// Later calls: one graph launch.  A shape whose capture fails stays on the eager path.
template <class Body>
ff_status run_replayed(ff_ctx* ctx, const ff_layer_desc* layers, const ff_layer_bufs* bufs, int n_layers, int B,
                       const void* extra, size_t extra_bytes, cudaStream_t st, Body run_body) {
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) {
    cudaGetLastError();
    return run_body(st);  // the caller is capturing already
  }
  std::vector<unsigned char> key;
  auto put = [&key](const void* p, size_t n) {
    const unsigned char* c = static_cast<const unsigned char*>(p);
    key.insert(key.end(), c, c + n);
  };
  const int route[3] = {ctx->gemm_path, ctx->tc.force_ncta, B};
  put(route, sizeof(route));
  put(&ctx->workspace, sizeof(void*));
  put(&ctx->workspace_bytes, sizeof(size_t));
  put(layers, sizeof(ff_layer_desc) * n_layers);
  put(bufs, sizeof(ff_layer_bufs) * n_layers);
  put(extra, extra_bytes);   // which entry point, and its further arguments that shape the launches

  ff_ctx::GraphEntry* ent = nullptr;
  for (auto& g : ctx->graphs)
    if (g.key == key) ent = &g;
  if (!ent) {
    if (ctx->graphs.size() >= FF_MAX_GRAPHS) {  // drop the entry unused for longest
      size_t old = 0;
      for (size_t i = 1; i < ctx->graphs.size(); ++i)
        if (ctx->graphs[i].last_use < ctx->graphs[old].last_use) old = i;
      if (ctx->graphs[old].exec) cudaGraphExecDestroy(ctx->graphs[old].exec);
      ctx->graphs.erase(ctx->graphs.begin() + old);
    }
    ctx->graphs.emplace_back();
    ctx->graphs.back().key = std::move(key);
    ctx->graphs.back().last_use = ++ctx->graph_clock;
    return run_body(st);
  }
  ent->last_use = ++ctx->graph_clock;
  if (ent->eager_only) return run_body(st);
  if (!ent->exec) {
    cudaError_t e;
    if (!ctx->capture_stream &&
        (e = cudaStreamCreateWithFlags(&ctx->capture_stream, cudaStreamNonBlocking)) != cudaSuccess) {
      ctx->capture_stream = nullptr;
      graph_gave_up(ctx, ent, "no capture stream", e);
      return run_body(st);
    }
    const uint64_t before = ctx->launches;
    if ((e = cudaStreamBeginCapture(ctx->capture_stream, cudaStreamCaptureModeThreadLocal)) != cudaSuccess) {
      graph_gave_up(ctx, ent, "capture did not start", e);
      return run_body(st);
    }
    // nothing runs while capturing: the launches are recorded on the library's own stream and replayed on the caller's
    const ff_status body = run_body(ctx->capture_stream);
    cudaGraph_t graph = nullptr;
    e = cudaStreamEndCapture(ctx->capture_stream, &graph);
    const uint64_t captured = ctx->launches - before;
    ctx->launches = before;
    cudaGraphExec_t exec = nullptr;
    if (body == FF_OK && e == cudaSuccess && graph) e = cudaGraphInstantiate(&exec, graph, 0);
    if (graph) cudaGraphDestroy(graph);
    if (body != FF_OK) {  // an argument the body rejects: nothing was launched
      ent->eager_only = true;
      cudaGetLastError();
      return body;
    }
    if (e != cudaSuccess || !exec) {
      graph_gave_up(ctx, ent, "capture or instantiation failed", e);
      return run_body(st);
    }
    ent->exec = exec;
    ent->launches = captured;
  }
  FF_CUDA(ctx, cudaGraphLaunch(ent->exec, st));
  ctx->launches += ent->launches;
  ctx->graph_replays++;
  return FF_OK;
}

ff_status train_step_graph(ff_ctx* ctx, const ff_layer_desc* layers, const ff_layer_bufs* bufs, int n_layers, int B,
                           float lambda, cudaStream_t st, int first) {
  const int tag[2] = {1, first};
  return run_replayed(ctx, layers, bufs, n_layers, B, tag, sizeof(tag), st, [&](cudaStream_t s) {
    return train_step_body(ctx, layers, bufs, n_layers, B, lambda, s, first);
  });
}

}  // namespace

// ================================================================================================
extern "C" {

ff_status ff_create(ff_ctx** out, int device) {
  if (!out) return FF_ERR_ARG;
  *out = nullptr;
  int n = 0;
  if (cudaGetDeviceCount(&n) != cudaSuccess || device < 0 || device >= n) return FF_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return FF_ERR_CUDA;
  if (prop.major != 10) return FF_ERR_UNSUPPORTED_ARCH;
  if (cudaSetDevice(device) != cudaSuccess) return FF_ERR_CUDA;
  ff_ctx* c = new (std::nothrow) ff_ctx();
  if (!c) return FF_ERR_ARG;
  c->device = device;
  c->sm_count = prop.multiProcessorCount;
  c->tc.sm_count = prop.multiProcessorCount;
  *out = c;
  return FF_OK;
}

ff_status ff_destroy(ff_ctx* ctx) {
  if (ctx) {
    for (auto& r : ctx->prof_recs) {
      cudaEventDestroy(r.a);
      cudaEventDestroy(r.b);
    }
    for (auto e : ctx->prof_pool) cudaEventDestroy(e);
    drop_graphs(ctx);
    if (ctx->capture_stream) cudaStreamDestroy(ctx->capture_stream);
  }
  delete ctx;
  return FF_OK;
}

ff_status ff_workspace_bytes(const ff_layer_desc* layers, int n_layers, int B, size_t* out_bytes) {
  if (!layers || n_layers <= 0 || B <= 0 || !out_bytes) return FF_ERR_ARG;
  size_t slab = 0;
  for (int l = 0; l < n_layers; ++l) {
    if (layers[l].K <= 0 || layers[l].N <= 0) return FF_ERR_ARG;
    const int sp = simt_wgrad_splits(layers[l], B, SIZE_MAX);
    size_t need = sp > 1 ? (size_t)sp * 2 * layers[l].N * layers[l].K * sizeof(int32_t) : 0;
    if (tc_update_supported(layers[l], B) && layers[l].kind == FF_CONV3X3) {
      // the larger of the single-CTA and CTA-pair split counts, so that either form finds room
      const int s1 = tc_conv_update_splits(layers[l], B, 0, 1), s2 = tc_conv_update_splits(layers[l], B, 0, 2);
      const size_t tc_need = tc_conv_update_slab_bytes(layers[l], s1 > s2 ? s1 : s2);
      if (tc_need > need) need = tc_need;
    }
    if (layers[l].kind == FF_CONV1X1 && tc_update_supported(layers[l], B)) {
      const int sp1 = tc_dense_slab_splits(layers[l].N, layers[l].K, (long long)B * layers[l].H * layers[l].Wd, 0);
      const size_t n1 = sp1 >= 2 ? (size_t)sp1 * 2 * layers[l].N * layers[l].K * sizeof(int32_t) : 0;
      if (n1 > need) need = n1;
    }
    if (layers[l].kind == FF_DWCONV3X3) need = (size_t)2 * layers[l].N * 9 * sizeof(int32_t) * dw_planes(layers[l], B);
    if (tc_im2col_ok(layers[l])) {
      const Im2colPlan pl = im2col_plan(layers[l], B, SIZE_MAX, 0);
      const size_t im_need = pl.slab_off - WS_BYTES + (size_t)pl.max_splits * pl.slab_bytes_per_split;
      if (im_need > need) need = im_need;
    }
    // a spatial layer of a split batch may be made to take two slabs so that its sums pass the range check
    if (layers[l].kind == FF_CONV3X3 || layers[l].kind == FF_CONV1X1) {
      const size_t two = (size_t)4 * layers[l].N * layers[l].K * sizeof(int32_t);
      if (two > need) need = two;
    }
    if (need < (size_t)2 * B * sizeof(float)) need = (size_t)2 * B * sizeof(float);   // per-sample normalisation factors
    if (layers[l].optimizer == FF_OPT_ADAM) need = up256(need) + adam_plane_bytes(layers[l]) + 256;  // sums plane at the tail
    if (need > slab) slab = need;
  }
  *out_bytes = WS_BYTES + (slab + 255) / 256 * 256;
  return FF_OK;
}

ff_status ff_set_workspace(ff_ctx* ctx, void* dev_ptr, size_t bytes) {
  if (!ctx) return FF_ERR_ARG;
  if (!dev_ptr || bytes < WS_BYTES) return fail(ctx, FF_ERR_WORKSPACE, "workspace too small");
  if (reinterpret_cast<uintptr_t>(dev_ptr) & 255) return fail(ctx, FF_ERR_ALIGN, "workspace must be 256-byte aligned");
  ctx->workspace = dev_ptr;
  ctx->workspace_bytes = bytes;
  ctx->status_zeroed = false;
  drop_graphs(ctx);
  return FF_OK;
}

ff_status ff_set_gemm_path(ff_ctx* ctx, int path) {
  if (!ctx) return FF_ERR_ARG;
  if (path != FF_GEMM_AUTO && path != FF_GEMM_SIMT && path != FF_GEMM_TENSOR) return fail(ctx, FF_ERR_ARG, "unknown gemm path");
  ctx->gemm_path = path;
  return FF_OK;
}

ff_status ff_set_tensor_form(ff_ctx* ctx, int ctas_per_tile) {
  if (!ctx) return FF_ERR_ARG;
  if (ctas_per_tile < 0 || ctas_per_tile > 2) return fail(ctx, FF_ERR_ARG, "ctas_per_tile must be 0, 1 or 2");
  ctx->tc.force_ncta = ctas_per_tile;
  return FF_OK;
}

ff_status ff_layer_forward(ff_ctx* ctx, const ff_layer_desc* layer, const ff_layer_bufs* bufs, int B, uint64_t step,
                           void* cuda_stream) {
  ff_status s = check_ctx(ctx);
  if (s != FF_OK) return s;
  if ((s = check_layer(ctx, layer, B)) != FF_OK) return s;
  if ((s = check_bufs(ctx, bufs, true)) != FF_OK) return s;
  if ((s = check_pitches(ctx, layer, bufs)) != FF_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if ((s = ensure_status(ctx, st)) != FF_OK) return s;
  FF_CUDA(ctx, cudaMemsetAsync(bufs->absmax, 0, FF_ABSMAX_LEN * sizeof(float), st));
  if ((s = set_step(ctx, step, 0.0f, false, st)) != FF_OK) return s;
  if ((s = quantize_input(ctx, *layer, *bufs, B, st)) != FF_OK) return s;
  if ((s = forward_from_xq(ctx, *layer, *bufs, B, nullptr, st)) != FF_OK) return s;
  return normalize_output(ctx, *layer, *bufs, B, nullptr, nullptr, st);
}

ff_status ff_layer_loss_grad(ff_ctx* ctx, const ff_layer_desc* layer, const ff_layer_bufs* bufs, int B,
                             const float* const* G_later, const float* theta_later, int n_later, float lambda,
                             uint64_t step, void* cuda_stream) {
  ff_status s = check_ctx(ctx);
  if (s != FF_OK) return s;
  if ((s = check_layer(ctx, layer, B)) != FF_OK) return s;
  if ((s = check_bufs(ctx, bufs, false)) != FF_OK) return s;
  if ((s = check_pitches(ctx, layer, bufs)) != FF_OK) return s;
  if (n_later < 0 || n_later > FF_MAX_LATER) return fail(ctx, FF_ERR_ARG, "n_later out of range");
  if (n_later > 0 && (!G_later || !theta_later)) return fail(ctx, FF_ERR_ARG, "G_later / theta_later is NULL");
  for (int j = 0; j < n_later; ++j)
    if (!G_later[j]) return fail(ctx, FF_ERR_ARG, "a G_later pointer is NULL");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if ((s = ensure_status(ctx, st)) != FF_OK) return s;
  if ((s = set_step(ctx, step, lambda, true, st)) != FF_OK) return s;
  return loss_grad_impl(ctx, *layer, *bufs, B, G_later, theta_later, n_later, lambda, st);
}

ff_status ff_layer_update(ff_ctx* ctx, const ff_layer_desc* layer, const ff_layer_bufs* bufs, int B, uint64_t step,
                          void* cuda_stream) {
  ff_status s = check_ctx(ctx);
  if (s != FF_OK) return s;
  if ((s = check_layer(ctx, layer, B)) != FF_OK) return s;
  if ((s = check_bufs(ctx, bufs, false)) != FF_OK) return s;
  if ((s = check_pitches(ctx, layer, bufs)) != FF_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if ((s = ensure_status(ctx, st)) != FF_OK) return s;
  if ((s = set_step(ctx, step, 0.0f, false, st)) != FF_OK) return s;  // Adam's update number is step + 1
  return run_update_gemm(ctx, *layer, *bufs, B, st);
}

ff_status ff_train_step_from(ff_ctx* ctx, const ff_layer_desc* layers, const ff_layer_bufs* bufs, int n_layers,
                             int first_trained, int B, float lambda, uint64_t step, void* cuda_stream) {
  ff_status s = check_ctx(ctx);
  if (s != FF_OK) return s;
  if ((s = check_layer_list(ctx, layers, bufs, n_layers, B)) != FF_OK) return s;
  if (first_trained < 0 || first_trained >= n_layers) return fail(ctx, FF_ERR_ARG, "first_trained out of range");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if ((s = ensure_status(ctx, st)) != FF_OK) return s;
  if ((s = set_step(ctx, step, lambda, true, st, bufs, n_layers)) != FF_OK) return s;
  if (ctx->graph_mode && !ctx->profiling) return train_step_graph(ctx, layers, bufs, n_layers, B, lambda, st, first_trained);
  return train_step_body(ctx, layers, bufs, n_layers, B, lambda, st, first_trained);
}

ff_status ff_train_step(ff_ctx* ctx, const ff_layer_desc* layers, const ff_layer_bufs* bufs, int n_layers, int B,
                        float lambda, uint64_t step, void* cuda_stream) {
  return ff_train_step_from(ctx, layers, bufs, n_layers, 0, B, lambda, step, cuda_stream);
}

int ff_dp_phase_count(int n_layers) { return n_layers > 0 ? 3 * n_layers + 2 : 0; }

ff_status ff_dp_train_phase(ff_ctx* ctx, const ff_layer_desc* layers, const ff_layer_bufs* bufs, int n_layers, int B_local,
                            int B_total, int row_offset, int phase, float lambda, uint64_t step, void* cuda_stream,
                            ff_dp_reduce* reduce, int* n_reduce) {
  ff_status s = check_ctx(ctx);
  if (s != FF_OK) return s;
  if (!reduce || !n_reduce) return fail(ctx, FF_ERR_ARG, "reduce / n_reduce is NULL");
  *n_reduce = 0;
  if ((s = check_layer_list(ctx, layers, bufs, n_layers, B_local)) != FF_OK) return s;
  if (B_total < B_local || row_offset < 0 || row_offset > B_total - B_local)
    return fail(ctx, FF_ERR_ARG, "rows [row_offset, row_offset + B_local) do not lie inside the batch of B_total");
  if (phase < 0 || phase >= ff_dp_phase_count(n_layers)) return fail(ctx, FF_ERR_ARG, "phase out of range");
  for (int l = 0; l < n_layers; ++l) {
    // counters, row counts and the INT32 weight-gradient range are those of the whole batch
    if ((s = check_layer(ctx, &layers[l], B_total)) != FF_OK) return s;
    if (l > 0 && bufs[l].X) return fail(ctx, FF_ERR_ARG, "a data-parallel step takes chained layers (X of layers > 0 NULL)");
    if (!bufs[l].accW_dump) return fail(ctx, FF_ERR_ARG, "a data-parallel step needs accW_dump of every layer");
    if (bufs[l].Skip) return fail(ctx, FF_ERR_ARG, "a data-parallel step takes no skip paths");
    if (layers[l].momentum != 0.0f && !bufs[l].Mom) return fail(ctx, FF_ERR_ARG, "momentum != 0 needs the buffer Mom");
    if (layers[l].optimizer == FF_OPT_ADAM && (!bufs[l].Mom || !bufs[l].Var))
      return fail(ctx, FF_ERR_ARG, "the Adam update needs the buffers Mom and Var");
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if ((s = ensure_status(ctx, st)) != FF_OK) return s;
  if ((s = set_step(ctx, step, lambda, true, st)) != FF_OK) return s;
  ctx->shard.B_total = B_total;
  ctx->shard.row_off = row_offset;
  ctx->shard.B_local = B_local;
  s = dp_phase_body(ctx, layers, bufs, n_layers, B_local, phase, lambda, st, reduce, n_reduce);
  ctx->shard.B_total = 0;
  ctx->shard.row_off = 0;
  ctx->shard.B_local = 0;
  ctx->accumulate_only = false;
  return s;
}

ff_status ff_set_graph_mode(ff_ctx* ctx, int on) {
  if (!ctx) return FF_ERR_ARG;
  if (on != 0 && on != 1) return fail(ctx, FF_ERR_ARG, "graph mode must be 0 or 1");
  ctx->graph_mode = on != 0;
  if (!on) drop_graphs(ctx);
  return FF_OK;
}

ff_status ff_predict(ff_ctx* ctx, const ff_layer_desc* layers, const ff_layer_bufs* bufs, int n_layers, int B, int n_classes,
                     int first_counted_layer, float* scores, int32_t* pred, uint64_t step, void* cuda_stream) {
  ff_status s = check_ctx(ctx);
  if (s != FF_OK) return s;
  if (n_classes <= 0) return fail(ctx, FF_ERR_ARG, "n_classes must be positive");
  if (B <= 0) return fail(ctx, FF_ERR_ARG, "B must be positive");
  if (((long long)n_classes * B) & 1) return fail(ctx, FF_ERR_ARG, "n_classes * B must be even (the candidate rows are processed as two halves)");
  if (!scores || !pred) return fail(ctx, FF_ERR_ARG, "scores / pred is NULL");
  if (!aligned16(scores) || !aligned16(pred)) return fail(ctx, FF_ERR_ALIGN, "scores / pred must be 16-byte aligned");
  if ((long long)n_classes * B / 2 >= (1LL << 30)) return fail(ctx, FF_ERR_RANGE, "too many candidate rows");
  const int half = n_classes * B / 2;  // rows of each of the two quantisation sets of the candidate batch
  if ((s = check_layer_list(ctx, layers, bufs, n_layers, half)) != FF_OK) return s;
  if (first_counted_layer < 0 || first_counted_layer >= n_layers) return fail(ctx, FF_ERR_ARG, "first_counted_layer out of range");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if ((s = ensure_status(ctx, st)) != FF_OK) return s;
  if ((s = set_step(ctx, step, 0.0f, false, st, bufs, n_layers)) != FF_OK) return s;
  auto body = [&](cudaStream_t sb) -> ff_status {
    ctx->joint_range = true;    // one quantiser range per tensor for the whole candidate batch
    ff_status r = forward_all(ctx, layers, bufs, n_layers, half, sb);
    ctx->joint_range = false;
    if (r != FF_OK) return r;
    LaterLayers gs;
    gs.n = n_layers - first_counted_layer;
    for (int j = 0; j < gs.n; ++j) {
      gs.G[j] = bufs[first_counted_layer + j].G;
      gs.theta[j] = 0.0f;
    }
    {
      ProfScope prof(ctx, FF_K_CLASSIFY, sb);
      classify_kernel<<<(B + EW_THREADS - 1) / EW_THREADS, EW_THREADS, 0, sb>>>(gs, B, n_classes, scores, pred);
    }
    FF_LAUNCH_CHECK(ctx);
    return FF_OK;
  };
  if (ctx->graph_mode && !ctx->profiling) {
    struct PredictKey {
      int tag, n_classes, first;
      float* scores;
      int32_t* pred;
    } extra;
    memset(&extra, 0, sizeof(extra));  // padding bytes are part of the key
    extra.tag = 2, extra.n_classes = n_classes, extra.first = first_counted_layer, extra.scores = scores, extra.pred = pred;
    return run_replayed(ctx, layers, bufs, n_layers, half, &extra, sizeof(extra), st, body);
  }
  return body(st);
}

ff_status ff_embed_labels(ff_ctx* ctx, const float* x, const int32_t* labels, int B, int n, int sets, int n_classes,
                          int label_stride, float on_value, float tau0, float eps, float* out, void* cuda_stream) {
  ff_status s = check_ctx(ctx);
  if (s != FF_OK) return s;
  if (!x || !labels || !out) return fail(ctx, FF_ERR_ARG, "x / labels / out is NULL");
  if (B <= 0 || n <= 0 || sets <= 0 || n_classes <= 0 || label_stride <= 0) return fail(ctx, FF_ERR_ARG, "sizes must be positive");
  if ((long long)(n_classes - 1) * label_stride >= n) return fail(ctx, FF_ERR_ARG, "the label places do not fit a sample");
  if (tau0 > 0.0f && !(eps >= 0.0f)) return fail(ctx, FF_ERR_ARG, "eps must be >= 0");
  if ((long long)sets * B * n >= (1LL << 40)) return fail(ctx, FF_ERR_RANGE, "output too large");
  if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(labels)) & 3)
    return fail(ctx, FF_ERR_ALIGN, "x / labels / out must be 4-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if ((s = ensure_status(ctx, st)) != FF_OK) return s;
  const int cap = ctx->sm_count * 8;
  embed_labels_kernel<<<B < cap ? B : cap, EMBED_THREADS, 0, st>>>(x, labels, B, n, sets, n_classes, label_stride, on_value,
                                                                  tau0, eps, out, status_ptr(ctx));
  FF_LAUNCH_CHECK(ctx);
  return FF_OK;
}

ff_status ff_poll_status(ff_ctx* ctx, void* cuda_stream) {
  ff_status s = check_ctx(ctx);
  if (s != FF_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  uint32_t h = 0;
  if (!ctx->status_zeroed) return FF_OK;
  FF_CUDA(ctx, cudaMemcpyAsync(&h, ctx->workspace, sizeof(h), cudaMemcpyDeviceToHost, st));
  FF_CUDA(ctx, cudaMemsetAsync(ctx->workspace, 0, sizeof(uint32_t), st));
  FF_CUDA(ctx, cudaStreamSynchronize(st));
  if (h & ST_TIMEOUT) {
    // a kernel that gave up may have left the loss kernels' completion tickets half counted: have the next call
    // clear the whole workspace header again
    ctx->status_zeroed = false;
    return fail(ctx, FF_ERR_DEVICE_TIMEOUT, "a bounded in-kernel wait ran out");
  }
  if (h & ST_NONFINITE) return fail(ctx, FF_ERR_NONFINITE, "a tensor to be quantised held Inf or NaN");
  if (h & ST_BADLABEL) return fail(ctx, FF_ERR_RANGE, "a label lay outside [0, n_classes)");
  if (h & ST_RANGE) return fail(ctx, FF_ERR_RANGE, "a weight-gradient sum left the INT32 range; that weight was not updated");
  return FF_OK;
}

ff_status ff_profile_start(ff_ctx* ctx) {
  if (!ctx) return FF_ERR_ARG;
  for (auto& r : ctx->prof_recs) {
    ctx->prof_pool.push_back(r.a);
    ctx->prof_pool.push_back(r.b);
  }
  ctx->prof_recs.clear();
  ctx->profiling = true;
  return FF_OK;
}

ff_status ff_profile_stop(ff_ctx* ctx, void* cuda_stream, float* ms_per_kernel, uint32_t* launches_per_kernel) {
  if (!ctx) return FF_ERR_ARG;
  if (!ms_per_kernel || !launches_per_kernel) return fail(ctx, FF_ERR_ARG, "output arrays are NULL");
  ctx->profiling = false;
  FF_CUDA(ctx, cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)));
  for (int k = 0; k < FF_K_COUNT; ++k) {
    ms_per_kernel[k] = 0.0f;
    launches_per_kernel[k] = 0;
  }
  for (auto& r : ctx->prof_recs) {
    float ms = 0.0f;
    FF_CUDA(ctx, cudaEventElapsedTime(&ms, r.a, r.b));
    ms_per_kernel[r.kid] += ms;
    launches_per_kernel[r.kid] += 1;
    ctx->prof_pool.push_back(r.a);
    ctx->prof_pool.push_back(r.b);
  }
  ctx->prof_recs.clear();
  return FF_OK;
}

ff_status ff_plan_wgrad(const ff_layer_desc* layer, int32_t B, int32_t sm_count, int32_t route, uint64_t workspace_bytes,
                        ff_wgrad_plan* out) {
  if (!layer || !out || B < 1 || sm_count < 1) return FF_ERR_ARG;
  const ff_layer_desc& L = *layer;
  if (L.kind != FF_CONV3X3 && L.kind != FF_CONV1X1 && L.kind != FF_LINEAR) return FF_ERR_ARG;
  const long long clen = (long long)B * rows_per_sample(L);   // contraction length: positions (rows) of one set
  memset(out, 0, sizeof(*out));
  if (route == FF_PLAN_TENSOR_SLABS) {
    // the split contraction of the tcgen05 kernels: work items per tile, consecutive splits sharing a slab
    if (L.kind == FF_LINEAR || !tc_update_supported(L, B)) return FF_ERR_ARG;
    const long long kblocks = L.kind == FF_CONV3X3 ? clen / 128 : (clen + 127) / 128;
    int splits = L.kind == FF_CONV3X3 ? tc_conv_update_splits(L, B, sm_count, 0)
                                      : tc_dense_slab_splits(L.N, L.K, clen, sm_count);
    if (splits < tc_min_splits(kblocks)) splits = tc_min_splits(kblocks);
    int per, kb_per_split;
    out->parts = tc_shared_slab_plan((int)kblocks, splits, &per, &kb_per_split);
    out->splits = (int)((kblocks + kb_per_split - 1) / kb_per_split);
    out->longest_register_sum = (long long)kb_per_split * 128;
    out->longest_part_sum = (long long)per * kb_per_split * 128;
    return FF_OK;
  }
  if (route == FF_PLAN_FIRST_LAYER) {
    if (!conv_small_ok(L.kind == FF_CONV3X3, L.Cin, L.N)) return FF_ERR_ARG;
    const ConvSmallWgradGeom g = conv_small_wgrad_plan(L, B, sm_count, false);
    out->parts = g.n_slabs;
    out->splits = g.n_slabs * g.blocks_per_plane;
    // a block strides through its plane's chunks; a plane holds chunks_per_slab chunks
    out->longest_register_sum = (long long)((g.chunks_per_slab + g.blocks_per_plane - 1) / g.blocks_per_plane) * CW_CHUNK;
    out->longest_part_sum = (long long)g.chunks_per_slab * CW_CHUNK;
    return FF_OK;
  }
  if (route == FF_PLAN_DP4A_SLABS) {
    int splits = simt_wgrad_splits(L, B, (size_t)workspace_bytes);
    if (splits < simt_min_splits(L, B)) return FF_ERR_WORKSPACE;
    const long long csplit = splits > 1 ? ((clen + splits - 1) / splits + SG_BK - 1) / SG_BK * SG_BK : clen;
    out->splits = splits > 1 ? simt_split_count((int)clen, splits) : 1;
    out->parts = out->splits;
    out->longest_register_sum = csplit;
    out->longest_part_sum = csplit;
    return FF_OK;
  }
  return FF_ERR_ARG;
}

ff_status ff_selftest_bounded_wait(ff_ctx* ctx, uint64_t limit_ns, void* cuda_stream) {
  ff_status s = check_ctx(ctx);
  if (s != FF_OK) return s;
  if (limit_ns == 0 || limit_ns > 1000000000ull) return fail(ctx, FF_ERR_ARG, "limit_ns must lie in [1, 1e9]");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if ((s = ensure_status(ctx, st)) != FF_OK) return s;
  bounded_wait_probe_kernel<<<1, 32, 0, st>>>(status_ptr(ctx), limit_ns);
  FF_LAUNCH_CHECK(ctx);
  return FF_OK;
}

const char* ff_last_error(const ff_ctx* ctx) { return ctx ? ctx->err : "context is NULL"; }

uint64_t ff_launch_count(const ff_ctx* ctx) { return ctx ? ctx->launches : 0; }

uint64_t ff_graph_replay_count(const ff_ctx* ctx) { return ctx ? ctx->graph_replays : 0; }

ff_status ff_int8_gemm(ff_ctx* ctx, const int8_t* A, const int8_t* Bm, int32_t* C, int M, int N, int K, int trans,
                       void* cuda_stream) {
  ff_status s = check_ctx(ctx);
  if (s != FF_OK) return s;
  if (!A || !Bm || !C || M <= 0 || N <= 0 || K <= 0) return fail(ctx, FF_ERR_ARG, "bad gemm arguments");
  if (!aligned16(A) || !aligned16(Bm) || !aligned16(C)) return fail(ctx, FF_ERR_ALIGN, "gemm pointers must be 16-byte aligned");
  if (K > ((1LL << 31) - 1) / (127LL * 127LL)) return fail(ctx, FF_ERR_RANGE, "contraction too long for INT32");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if ((s = ensure_status(ctx, st)) != FF_OK) return s;
  bool tc_ok = tc_gemm_supported(M, N, K, trans);
  if (ctx->gemm_path == FF_GEMM_TENSOR && !tc_ok) return fail(ctx, FF_ERR_ARG, "shape not supported by the tensor-core gemm");
  if (tc_ok && ctx->gemm_path != FF_GEMM_SIMT) {
    ProfScope prof(ctx, FF_K_RAW_GEMM, st);
    s = tc_gemm(ctx->tc, A, Bm, C, M, N, K, trans, status_ptr(ctx), st);
    if (s != FF_OK) return fail(ctx, s, "tensor-core gemm launch failed: %s", ctx->tc.err);
    ctx->launches++;
    return FF_OK;
  }
  RawEpilogue epi{C, M, N};
  if (!trans) return launch_simt<DenseView, DenseView, false, 1>(ctx, dense(A, M, K), dense(Bm, N, K), M, N, K, epi, st);
  return launch_simt<DenseView, DenseView, true, 1>(ctx, dense(A, K, M), dense(Bm, K, N), M, N, K, epi, st);
}

// ------------------------------------------------------------------------------------------------
// ff_loss_coef_static: the loss / coefficient kernel with its partial-sum scratch in a fixed device
// array instead of the caller's workspace.
//
// The array below is part of the library image: every GPU that loads the library holds these few
// kilobytes until the process exits.  In host code the name `g_static_loss_scratch` is only a handle;
// the device address the kernel needs comes from cudaGetSymbolAddress, asked for once per device
// while that device is current.
// ------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_loss_scratch[sizeof(LossScratch)];
static_assert(FF_STATIC_LOSS_MAX_SAMPLES == LOSS_MAX_BLOCKS * LOSS_THREADS, "one scratch slot per block of LOSS_THREADS samples");

namespace {
constexpr int STATIC_MAX_DEVICES = 64;
LossScratch* g_static_loss_ptr[STATIC_MAX_DEVICES] = {nullptr};
std::mutex g_static_loss_mutex;  // guards the table above (first calls from several host threads)

void static_err(char* err, size_t err_len, const char* msg, const char* detail = "") {
  if (err && err_len) snprintf(err, err_len, "%s%s", msg, detail);
}
}  // namespace

ff_status ff_loss_coef_static(const float* G, float theta, const float* const* G_later, const float* theta_later, int n_later,
                              float lambda, int B, const int32_t* rowmax, float* absmax, float* coef, float* loss,
                              void* cuda_stream, char* err, size_t err_len) {
  if (!G || !rowmax || !absmax || !coef || !loss) {
    static_err(err, err_len, "a required device pointer is NULL");
    return FF_ERR_ARG;
  }
  if (B <= 0) {
    static_err(err, err_len, "B must be positive");
    return FF_ERR_ARG;
  }
  if (2LL * B > FF_STATIC_LOSS_MAX_SAMPLES) {
    static_err(err, err_len, "2*B exceeds FF_STATIC_LOSS_MAX_SAMPLES, the size the built-in scratch array was laid out for");
    return FF_ERR_RANGE;
  }
  if (n_later < 0 || n_later > FF_MAX_LATER || (n_later > 0 && (!G_later || !theta_later))) {
    static_err(err, err_len, "bad list of later layers");
    return FF_ERR_ARG;
  }
  LaterLayers later;
  later.n = n_later;
  for (int j = 0; j < n_later; ++j) {
    if (!G_later[j]) {
      static_err(err, err_len, "a G_later pointer is NULL");
      return FF_ERR_ARG;
    }
    later.G[j] = G_later[j];
    later.theta[j] = theta_later[j];
  }
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) {
    static_err(err, err_len, "cudaGetDevice: ", e != cudaSuccess ? cudaGetErrorString(e) : "device index out of range");
    return FF_ERR_CUDA;
  }
  LossScratch* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_loss_mutex);
    if (!g_static_loss_ptr[dev]) {
      // first call on this device: turn the symbol into the address of this device's copy of the array
      void* ptr = nullptr;
      e = cudaGetSymbolAddress(&ptr, g_static_loss_scratch);
      if (e != cudaSuccess || !ptr) {
        static_err(err, err_len, "cudaGetSymbolAddress: ", cudaGetErrorString(e));
        return FF_ERR_CUDA;
      }
      g_static_loss_ptr[dev] = static_cast<LossScratch*>(ptr);
    }
    scratch = g_static_loss_ptr[dev];
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // the array keeps whatever the last call left: the block-completion ticket has to start at zero
  e = cudaMemsetAsync(&scratch->ticket, 0, sizeof(scratch->ticket), st);
  if (e != cudaSuccess) {
    static_err(err, err_len, "cudaMemsetAsync: ", cudaGetErrorString(e));
    return FF_ERR_CUDA;
  }
  const int blocks = (2 * B + LOSS_THREADS - 1) / LOSS_THREADS;  // <= LOSS_MAX_BLOCKS by the size check above
  loss_coef_kernel<<<blocks, LOSS_THREADS, 0, st>>>(G, theta, later, lambda, B, rowmax, absmax, coef, loss, scratch);
  e = cudaGetLastError();
  if (e != cudaSuccess) {
    static_err(err, err_len, "launch: ", cudaGetErrorString(e));
    return FF_ERR_CUDA;
  }
  return FF_OK;
}

}  // extern "C"
