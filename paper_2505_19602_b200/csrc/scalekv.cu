// Host runtime and C ABI of the ScaleKV hot path (see include/scalekv.h for the contract).
// The context plans the paged store, tracks the per-layer call order and lengths, orders the two
// streams with events and launches the kernels.  Nothing here computes on the CPU.
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include "../../include/scalekv.h"
#include "attend_tc.cuh"
#include "kernels_simt.cuh"

using namespace scalekv;

namespace {

// Layers l, l + kSets, l + 2 kSets, ... share one transient page set and one buffer of recorded window logits: the
// part of a current map beyond a layer's persistent capacity only lives from that layer's attend to its compress,
// and with four sets the compress of layer l has the attends of three more layers to hide under before layer
// l + 4 needs the set back (with two, the chain attend(l) -> compress(l) -> attend(l + 2) bounds the scales whose
// kernels are short).
constexpr int kSets = 4;
// layer_stats splits a slice's keys over several CTAs while the launch would otherwise leave SMs idle; this many CTAs
// bound the scratch of their partial results (about 10 MB)
constexpr int kStatsMaxCtas = 592;
constexpr int kNumClasses = 7;
enum KernelClass { kAppend = 0, kAttend = 1, kScore = 2, kSelect = 3, kCompact = 4, kOther = 5, kCompress = 6 };

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct LayerPlan {
  int cap = 0;            // largest cache a compress can leave behind
  int max_len = 0;        // largest cache during any step
  int persist_pages = 0;  // pages owned by each slice of this layer
  int total_pages = 0;    // logical pages per slice (persistent + transient)
  size_t page_table_off = 0;  // element offset into the page-table area
  int first_page = 0;         // first persistent page id
};

struct Plan {
  int n_layers, B, H, d, esize, K, P, page_shift, n_slices, max_window;
  std::vector<int> n, N;            // tokens per scale, cumulative (N[0] = 0)
  std::vector<int> budgets;         // [layers][K]
  std::vector<std::vector<int>> windows;   // per scale: rows whose logits attend records (empty: none)
  std::vector<LayerPlan> layers;
  int trans_pages_per_slice = 0;    // size of one transient set per slice
  int trans_first[kSets] = {0, 0, 0, 0};
  long long n_pages = 0;
  int ld_s = 0;                     // padded max length (leading dimension of per-slice scratch)
  int ld_l = 0;                     // leading dimension of a logit row: room for the history rounded up to a key tile and a ragged last tile
  int n_max = 0;
  // pool layout (byte offsets)
  size_t off_k, off_v, off_pos, off_pt, off_len, off_status, pool_bytes;
  size_t pt_elems, logits_elems;
  // workspace layout
  size_t off_logits, off_wlse, off_scores, off_keys, off_keep, off_kept, off_hbud, off_acc, off_stats, ws_bytes;
};

// Raster indices of the observation window of an h x w map (see scalekv_window_centroids).
std::vector<int> centroid_window(int h, int w, int n_patches) {
  std::vector<int> out;
  if ((long long)h * w <= n_patches) {
    for (int i = 0; i < h * w; ++i) out.push_back(i);
    return out;
  }
  int g = (int)std::floor(std::sqrt((double)n_patches));
  while ((g + 1) * (g + 1) <= n_patches) ++g;
  while (g * g > n_patches) --g;
  for (int a = 0; a < g; ++a) {
    const int r0 = (int)((long long)a * h / g), r1 = (int)((long long)(a + 1) * h / g);
    if (r1 <= r0) continue;
    for (int b = 0; b < g; ++b) {
      const int c0 = (int)((long long)b * w / g), c1 = (int)((long long)(b + 1) * w / g);
      if (c1 <= c0) continue;
      out.push_back(((r0 + r1 - 1) / 2) * w + (c0 + c1 - 1) / 2);
    }
  }
  std::sort(out.begin(), out.end());
  out.erase(std::unique(out.begin(), out.end()), out.end());
  return out;
}

scalekv_status make_plan(const scalekv_config *c, Plan &p, std::string &err) {
  if (!c || !c->scale_h || !c->scale_w || !c->budgets) { err = "null config field"; return SCALEKV_ERR_INVALID_ARG; }
  if (c->n_layers < 1 || c->batch < 1 || c->n_heads < 1 || c->n_scales < 1 || c->n_scales > SCALEKV_MAX_SCALES) {
    err = "n_layers, batch, n_heads >= 1 and 1 <= n_scales <= 32 required"; return SCALEKV_ERR_INVALID_ARG;
  }
  if (c->max_window < 1 || c->max_window > SCALEKV_MAX_WINDOW) { err = "max_window out of range"; return SCALEKV_ERR_INVALID_ARG; }
  if (!((c->dtype == SCALEKV_BF16 && c->head_dim == 128) || (c->dtype == SCALEKV_F32 && c->head_dim == 64))) {
    err = "unsupported (dtype, head_dim): bf16 x 128 and f32 x 64 are built"; return SCALEKV_ERR_UNSUPPORTED;
  }
  p.n_layers = c->n_layers; p.B = c->batch; p.H = c->n_heads; p.d = c->head_dim;
  p.esize = c->dtype == SCALEKV_BF16 ? 2 : 4;
  p.K = c->n_scales; p.max_window = c->max_window;
  p.P = c->page_tokens == 0 ? 128 : c->page_tokens;
  if (p.P < 16 || (p.P & (p.P - 1))) { err = "page_tokens must be a power of two >= 16"; return SCALEKV_ERR_INVALID_ARG; }
  p.page_shift = 0; while ((1 << p.page_shift) < p.P) ++p.page_shift;
  p.n_slices = p.B * p.H;
  p.n.resize(p.K); p.N.assign(p.K + 1, 0);
  p.n_max = 0;
  for (int k = 0; k < p.K; ++k) {
    if (c->scale_h[k] < 1 || c->scale_w[k] < 1) { err = "scale sides must be >= 1"; return SCALEKV_ERR_INVALID_ARG; }
    p.n[k] = c->scale_h[k] * c->scale_w[k];
    p.N[k + 1] = p.N[k] + p.n[k];
    p.n_max = std::max(p.n_max, p.n[k]);
  }
  p.budgets.assign(c->budgets, c->budgets + (size_t)p.n_layers * p.K);
  if (c->window_patches < 0 || c->window_patches > c->max_window) { err = "window_patches must lie in [0, max_window]"; return SCALEKV_ERR_INVALID_ARG; }
  p.windows.assign(p.K, std::vector<int>());
  if (c->window_kind != SCALEKV_WINDOW_CENTROIDS && c->window_kind != SCALEKV_WINDOW_LAST) { err = "unknown window_kind"; return SCALEKV_ERR_INVALID_ARG; }
  if (c->window_patches > 0)
    for (int k = 0; k < p.K; ++k) {
      if (c->window_kind == SCALEKV_WINDOW_LAST) {
        const int m = std::min(c->window_patches, p.n[k]);
        for (int i = 0; i < m; ++i) p.windows[k].push_back(p.n[k] - m + i);
      } else {
        p.windows[k] = centroid_window(c->scale_h[k], c->scale_w[k], c->window_patches);
      }
    }
  p.layers.resize(p.n_layers);
  int trans_max = 0, len_max = 0;
  size_t pt = 0;
  long long page = 0;
  for (int l = 0; l < p.n_layers; ++l) {
    LayerPlan &lp = p.layers[l];
    int hist = 0;
    for (int k = 0; k < p.K; ++k) {
      const int L = hist + p.n[k];
      lp.max_len = std::max(lp.max_len, L);
      const int bud = p.budgets[(size_t)l * p.K + k];
      if (bud < SCALEKV_KEEP_ALL) { err = "budget < -1"; return SCALEKV_ERR_INVALID_ARG; }
      const int wmax = std::min(p.max_window, p.n[k]);
      const long long kept = bud == SCALEKV_KEEP_ALL ? L : std::min<long long>(L, (long long)bud + wmax);
      hist = (int)kept;
      lp.cap = std::max(lp.cap, hist);
    }
    lp.total_pages = (lp.max_len + p.P - 1) / p.P;
    lp.persist_pages = std::min(lp.total_pages, (lp.cap + p.P - 1) / p.P);
    lp.page_table_off = pt;
    pt += (size_t)p.n_slices * lp.total_pages;
    lp.first_page = (int)page;
    page += (long long)p.n_slices * lp.persist_pages;
    trans_max = std::max(trans_max, lp.total_pages - lp.persist_pages);
    len_max = std::max(len_max, lp.max_len);
  }
  p.trans_pages_per_slice = trans_max;
  for (int t = 0; t < kSets; ++t) { p.trans_first[t] = (int)page; page += (long long)p.n_slices * trans_max; }
  if (page > 0x7fffffffLL / p.P) { err = "store too large for 32-bit row indices"; return SCALEKV_ERR_CAPACITY; }
  p.n_pages = page;
  p.pt_elems = pt;
  p.ld_s = (int)align_up((size_t)len_max, 64);
  p.ld_l = (int)align_up((size_t)len_max + 256, 64);
  const size_t row_bytes = (size_t)p.d * p.esize;
  size_t o = 0;
  p.off_k = o; o = align_up(o + (size_t)p.n_pages * p.P * row_bytes, 1024);
  p.off_v = o; o = align_up(o + (size_t)p.n_pages * p.P * row_bytes, 1024);
  p.off_pos = o; o = align_up(o + (size_t)p.n_pages * p.P * 4, 1024);
  p.off_pt = o; o = align_up(o + pt * 4, 1024);
  p.off_len = o; o = align_up(o + (size_t)p.n_layers * p.n_slices * 4, 1024);
  p.off_status = o; o = align_up(o + 256, 1024);
  p.pool_bytes = o;
  o = 0;
  p.logits_elems = (size_t)p.n_slices * p.max_window * p.ld_l;   // one buffer per set
  p.off_logits = o; o = align_up(o + kSets * p.logits_elems * 4, 1024);
  p.off_wlse = o; o = align_up(o + kSets * (size_t)p.n_slices * p.max_window * 4, 1024);   // one per set
  p.off_scores = o; o = align_up(o + (size_t)p.n_slices * p.ld_s * 4, 1024);
  p.off_keys = o; o = align_up(o + (size_t)p.n_slices * p.ld_s * 4, 1024);
  p.off_keep = o; o = align_up(o + (size_t)p.n_slices * p.ld_s * 4, 1024);
  p.off_kept = o; o = align_up(o + (size_t)p.n_slices * 4, 1024);
  p.off_hbud = o; o = align_up(o + (size_t)p.n_slices * 4, 1024);
  p.off_acc = o; o = align_up(o + 16 + (size_t)p.n_slices * 16, 1024);
  p.off_stats = o; o = align_up(o + (size_t)kStatsMaxCtas * 64 * kStatsRec * 4, 1024);   // key-range partials of layer_stats
  p.ws_bytes = o;
  return SCALEKV_OK;
}

}  // namespace

struct scalekv_ctx {
  Plan plan;
  int device = 0;
  int dtype = 0;
  float scale = 0.f;
  char *pool = nullptr, *ws = nullptr;
  cudaStream_t s_main = nullptr, s_side = nullptr;
  cudaEvent_t ev_join = nullptr;   // scalekv_join: marks the side stream's progress
  // scalekv_step_host only: copy streams of the library's own and, per staging half, the events that chain them
  cudaStream_t s_h2d = nullptr, s_d2h = nullptr;
  cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr}, ev_att[2] = {nullptr, nullptr};
  int set_layer[2] = {-1, -1};     // layer that last used a staging half (-1: unused)
  long long host_steps = 0;
  std::vector<int> page_table_host;
  // per layer state
  std::vector<int> next_scale;     // scale expected by the next append
  std::vector<int> hist;           // entries before the current map (uniform over slices)
  std::vector<int> pending;        // n_k of an appended, not yet committed current map (0 = none)
  std::vector<int> attended;       // attend ran for the pending map
  std::vector<char> in_store;      // the pending map's rows have been copied into the pages
  std::vector<char> logits_padded; // attend recorded the logits while the current map was still outside the store
  std::vector<int> logits_of;      // scale whose window logits attend recorded for this layer (-1: none)
  std::vector<scalekv_tensor> pend_k, pend_v;   // the caller's tensors of a pending map that is not in the store yet
  std::vector<cudaEvent_t> ev_attend, ev_compress;
  std::vector<char> ev_compress_live;
  std::vector<char> ev_compress_joined;   // stream_main has already waited for that compress (scalekv_join)
  std::vector<char> map_lost;      // the layer's last map was attended and its transient rows then given to another layer
  bool fused_ok = false;           // a slice's keys and keep list fit one CTA's shared memory: compress is one launch
  bool select_smem_ok = false;     // the separate select kernel can stage a slice's keys in shared memory
  bool compact_smem_ok = false;    // the separate compact kernel can stage a slice's keep list in shared memory
  size_t fused_smem = 0;
  bool side_dirty = false;         // stream_side has work that stream_main has not joined yet
  int set_owner[kSets] = {-1, -1, -1, -1};   // layer that last appended into each transient page set / logit buffer
  int64_t launches = 0;
  int scores_len = 0;              // length of the score vectors left by the last evicting compress
  bool profile = false;            // launches are bracketed by events
  bool serialize = false;          // compress runs on stream_main (every kernel timed alone)
  struct Timed { cudaEvent_t a, b; int cls; };
  std::vector<Timed> timed;
  std::vector<cudaEvent_t> event_pool;
  double prof_ms[kNumClasses] = {0};
  int64_t prof_n[kNumClasses] = {0};
  std::string err = "ok";
  AttendTc tc;
};

namespace {

scalekv_status fail(scalekv_ctx *c, scalekv_status st, const char *fmt, ...) {
  char buf[512];
  va_list ap; va_start(ap, fmt); vsnprintf(buf, sizeof buf, fmt, ap); va_end(ap);
  if (c) c->err = buf;
  return st;
}

#define CU(call)                                                                                   \
  do {                                                                                             \
    cudaError_t e_ = (call);                                                                       \
    if (e_ != cudaSuccess) return fail(ctx, SCALEKV_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

LayerView layer_view(scalekv_ctx *c, int l) {
  const Plan &p = c->plan;
  LayerView lv;
  lv.k_pool = c->pool + p.off_k;
  lv.v_pool = c->pool + p.off_v;
  lv.pos_pool = reinterpret_cast<int *>(c->pool + p.off_pos);
  lv.page_table = reinterpret_cast<const int *>(c->pool + p.off_pt) + p.layers[l].page_table_off;
  lv.hist_len = reinterpret_cast<int *>(c->pool + p.off_len) + (size_t)l * p.n_slices;
  lv.status = reinterpret_cast<int *>(c->pool + p.off_status);
  lv.pages_per_slice = p.layers[l].total_pages;
  lv.page_shift = p.page_shift;
  lv.page_mask = p.P - 1;
  lv.row_bytes = p.d * p.esize;
  lv.n_slices = p.n_slices;
  lv.n_heads = p.H;
  return lv;
}

TensorView tview(const scalekv_tensor &t) {
  TensorView v; v.ptr = static_cast<const char *>(t.ptr); v.sb = t.stride_b; v.sh = t.stride_h; v.st = t.stride_t;
  return v;
}

bool tensor_ok(const scalekv_tensor &t, int esize) {
  if (!t.ptr) return false;
  if (reinterpret_cast<uintptr_t>(t.ptr) & 15) return false;
  return ((t.stride_b * esize) % 16 == 0) && ((t.stride_h * esize) % 16 == 0) && ((t.stride_t * esize) % 16 == 0);
}

const char *const kClassNames[kNumClasses] = {"scalekv.append", "scalekv.attend", "scalekv.score", "scalekv.select",
                                               "scalekv.compact", "scalekv.other", "scalekv.compress"};

struct Scope {  // brackets one launch with an NVTX range and, when profiling, with events; counts launches
  scalekv_ctx *c; cudaStream_t s; int cls; cudaEvent_t a = nullptr, b = nullptr;
  Scope(scalekv_ctx *c_, cudaStream_t s_, int cls_) : c(c_), s(s_), cls(cls_) {
    nvtxRangePushA(kClassNames[cls]);
    if (c->profile) {
      a = take(); b = take();
      if (a && b) cudaEventRecord(a, s);
    }
  }
  cudaEvent_t take() {
    if (!c->event_pool.empty()) { cudaEvent_t e = c->event_pool.back(); c->event_pool.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); return nullptr; }   // this launch goes untimed
    return e;
  }
  ~Scope() {
    nvtxRangePop();
    c->launches++;
    if (c->profile) {
      if (a && b) { cudaEventRecord(b, s); c->timed.push_back({a, b, cls}); }
      else { if (a) c->event_pool.push_back(a); if (b) c->event_pool.push_back(b); }
    }
  }
};

void drain_profile(scalekv_ctx *c) {
  for (auto &t : c->timed) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, t.a, t.b) == cudaSuccess) { c->prof_ms[t.cls] += ms; c->prof_n[t.cls]++; }
    c->event_pool.push_back(t.a); c->event_pool.push_back(t.b);
  }
  c->timed.clear();
}

// Raises a kernel's dynamic shared-memory limit; false when the device cannot give that much.
template <typename F> bool set_smem(F *f, size_t bytes) {
  if (bytes > (size_t)0x7fffffff) return false;
  if (cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) == cudaSuccess) return true;
  cudaGetLastError();
  return false;
}

scalekv_status check_launch(scalekv_ctx *ctx, const char *what) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ctx, SCALEKV_ERR_CUDA, "launch of %s failed: %s", what, cudaGetErrorString(e));
  return SCALEKV_OK;
}

// Copies a pending current map that still lives in the caller's tensors into the pages (stream_main).
// The tensor-core attend does this itself while it streams the map; this kernel serves every other
// order of calls (compress, statistics or export without a preceding attend).
scalekv_status materialize(scalekv_ctx *ctx, int l) {
  if (ctx->pending[l] == 0 || ctx->in_store[l]) return SCALEKV_OK;
  const Plan &p = ctx->plan;
  const int k = ctx->next_scale[l] - 1;
  const int nk = ctx->pending[l];
  {
    Scope sc(ctx, ctx->s_main, kAppend);
    dim3 grid((nk + 63) / 64, p.n_slices);
    append_kernel<<<grid, 256, 0, ctx->s_main>>>(layer_view(ctx, l), tview(ctx->pend_k[l]), tview(ctx->pend_v[l]), nk, p.N[k], p.esize);
  }
  ctx->in_store[l] = 1;
  return check_launch(ctx, "append");
}

scalekv_status commit_pending(scalekv_ctx *ctx, int l, cudaStream_t s) {
  if (ctx->pending[l] == 0) return SCALEKV_OK;
  const Plan &p = ctx->plan;
  if (!ctx->in_store[l]) return fail(ctx, SCALEKV_ERR_BAD_STATE, "layer %d: pending map is not in the store", l);
  const int L = ctx->hist[l] + ctx->pending[l];
  if (L > p.layers[l].persist_pages * p.P && p.layers[l].persist_pages < p.layers[l].total_pages)
    return fail(ctx, SCALEKV_ERR_CAPACITY, "layer %d: %d entries kept without compress exceed the persistent capacity %d",
                l, L, p.layers[l].persist_pages * p.P);
  {
    Scope sc(ctx, s, kOther);
    commit_kernel<<<(p.n_slices + 255) / 256, 256, 0, s>>>(layer_view(ctx, l), ctx->pending[l]);
  }
  ctx->hist[l] = L;
  ctx->pending[l] = 0;
  ctx->attended[l] = 0;
  return check_launch(ctx, "commit");
}

scalekv_status fill_window(scalekv_ctx *ctx, int l, int w, const int32_t *window_pos, WindowArg &wa) {
  const Plan &p = ctx->plan;
  const int k = ctx->next_scale[l] - 1;
  wa.n_prev = p.N[k];
  wa.n_k = p.n[k];
  if (window_pos == nullptr) {
    if (wa.n_k > p.max_window) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "whole-map window needs n_k <= max_window");
    wa.w = wa.n_k; wa.all = 1;
    for (int j = 0; j < wa.w; ++j) wa.pos[j] = j;
  } else {
    if (w < 1 || w > p.max_window || w > wa.n_k) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "window size %d out of range", w);
    wa.w = w; wa.all = 0;
    for (int j = 0; j < w; ++j) {
      if (window_pos[j] < 0 || window_pos[j] >= wa.n_k || (j > 0 && window_pos[j] <= window_pos[j - 1]))
        return fail(ctx, SCALEKV_ERR_INVALID_ARG, "window_pos must be ascending, distinct and inside the current map");
      wa.pos[j] = window_pos[j];
    }
  }
  for (int j = wa.w; j < kMaxWindow; ++j) wa.pos[j] = 0x7fffffff;
  return SCALEKV_OK;
}

}  // namespace

extern "C" {

scalekv_status scalekv_query_sizes(const scalekv_config *cfg, size_t *pool_bytes, size_t *workspace_bytes) {
  Plan p; std::string err;
  scalekv_status st = make_plan(cfg, p, err);
  if (st != SCALEKV_OK) return st;
  if (pool_bytes) *pool_bytes = p.pool_bytes;
  if (workspace_bytes) *workspace_bytes = p.ws_bytes;
  return SCALEKV_OK;
}

scalekv_status scalekv_init(const scalekv_config *cfg, scalekv_ctx **out) {
  if (!out) return SCALEKV_ERR_INVALID_ARG;
  *out = nullptr;
  scalekv_ctx *ctx = new scalekv_ctx();
  std::string err;
  scalekv_status st = make_plan(cfg, ctx->plan, err);
  if (st != SCALEKV_OK) { delete ctx; return st; }
  const Plan &p = ctx->plan;
  if (!cfg->pool || !cfg->workspace) { delete ctx; return SCALEKV_ERR_INVALID_ARG; }
  if (cfg->pool_bytes < p.pool_bytes || cfg->workspace_bytes < p.ws_bytes) { delete ctx; return SCALEKV_ERR_CAPACITY; }
  if ((reinterpret_cast<uintptr_t>(cfg->pool) & 1023) || (reinterpret_cast<uintptr_t>(cfg->workspace) & 255)) {
    delete ctx; return SCALEKV_ERR_INVALID_ARG;
  }
  ctx->device = cfg->device; ctx->dtype = cfg->dtype;
  ctx->scale = cfg->softmax_scale != 0.f ? cfg->softmax_scale : 1.0f / std::sqrt((float)cfg->head_dim);
  ctx->pool = static_cast<char *>(cfg->pool); ctx->ws = static_cast<char *>(cfg->workspace);
  ctx->s_main = static_cast<cudaStream_t>(cfg->stream_main);
  ctx->s_side = cfg->stream_side ? static_cast<cudaStream_t>(cfg->stream_side) : ctx->s_main;
  auto bail = [&](scalekv_status s) {     // a failed init gives back what it had created so far
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    for (auto e : ctx->ev_attend) if (e) cudaEventDestroy(e);
    for (auto e : ctx->ev_compress) if (e) cudaEventDestroy(e);
    delete ctx;
    return s;
  };
  if (cudaSetDevice(cfg->device) != cudaSuccess) return bail(SCALEKV_ERR_CUDA);
  if (cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming) != cudaSuccess) return bail(SCALEKV_ERR_CUDA);
  int major = 0, minor = 0;
  cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, cfg->device);
  cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, cfg->device);
  if (major != 10) return bail(SCALEKV_ERR_UNSUPPORTED);
  // page tables: persistent pages first, then the transient set the layer shares (layer mod kSets)
  ctx->page_table_host.resize(p.pt_elems);
  for (int l = 0; l < p.n_layers; ++l) {
    const LayerPlan &lp = p.layers[l];
    for (int s = 0; s < p.n_slices; ++s)
      for (int j = 0; j < lp.total_pages; ++j) {
        int page = j < lp.persist_pages
                       ? lp.first_page + s * lp.persist_pages + j
                       : p.trans_first[l % kSets] + s * p.trans_pages_per_slice + (j - lp.persist_pages);
        ctx->page_table_host[lp.page_table_off + (size_t)s * lp.total_pages + j] = page;
      }
  }
  if (cudaMemcpy(ctx->pool + p.off_pt, ctx->page_table_host.data(), p.pt_elems * 4, cudaMemcpyHostToDevice) != cudaSuccess)
    return bail(SCALEKV_ERR_CUDA);
  // pages start out as zeros: tiles are loaded whole, and rows beyond a slice's length must be finite
  if (cudaMemset(ctx->pool + p.off_k, 0, p.off_pos - p.off_k) != cudaSuccess) return bail(SCALEKV_ERR_CUDA);
  if (cudaMemset(ctx->pool + p.off_len, 0, (size_t)p.n_layers * p.n_slices * 4) != cudaSuccess) return bail(SCALEKV_ERR_CUDA);
  if (cudaMemset(ctx->pool + p.off_status, 0, 256) != cudaSuccess) return bail(SCALEKV_ERR_CUDA);
  ctx->next_scale.assign(p.n_layers, 0);
  ctx->hist.assign(p.n_layers, 0);
  ctx->pending.assign(p.n_layers, 0);
  ctx->attended.assign(p.n_layers, 0);
  ctx->in_store.assign(p.n_layers, 1);
  ctx->logits_of.assign(p.n_layers, -1);
  ctx->logits_padded.assign(p.n_layers, 0);
  ctx->pend_k.resize(p.n_layers); ctx->pend_v.resize(p.n_layers);
  ctx->ev_attend.resize(p.n_layers); ctx->ev_compress.resize(p.n_layers);
  ctx->ev_compress_live.assign(p.n_layers, 0);
  ctx->ev_compress_joined.assign(p.n_layers, 0);
  ctx->map_lost.assign(p.n_layers, 0);
  for (int l = 0; l < p.n_layers; ++l) {
    if (cudaEventCreateWithFlags(&ctx->ev_attend[l], cudaEventDisableTiming) != cudaSuccess) return bail(SCALEKV_ERR_CUDA);
    if (cudaEventCreateWithFlags(&ctx->ev_compress[l], cudaEventDisableTiming) != cudaSuccess) return bail(SCALEKV_ERR_CUDA);
  }
  {
    // every kernel that sizes its shared memory from the schedule is checked now, so that a configuration the
    // kernels cannot take is refused here and not at its first launch
    bool ok = true;
    if (cfg->dtype == SCALEKV_BF16) {
      ok = ok && set_smem(attend_simt_kernel<__nv_bfloat16, 128>, (64 * 132 * 2 + 64 * 65 + 192) * 4);
      ok = ok && set_smem(score_logits_kernel<__nv_bfloat16, 128>, 2 * 64 * 132 * 4);
      ok = ok && set_smem(layer_stats_kernel<__nv_bfloat16, 128>, layer_stats_smem_bytes<128>(64));
    } else {
      ok = ok && set_smem(layer_stats_kernel<float, 64>, layer_stats_smem_bytes<64>(64));
      ok = ok && set_smem(attend_simt_kernel<float, 64>, (64 * 68 * 2 + 64 * 65 + 192) * 4);
      ok = ok && set_smem(score_logits_kernel<float, 64>, 2 * 64 * 68 * 4);
    }
    // select and compact stage a slice in shared memory when it fits and work from global memory when it does not
    int max_pages = 0;
    for (const LayerPlan &lp : p.layers) max_pages = std::max(max_pages, lp.total_pages);
    ctx->select_smem_ok = set_smem(select_kernel, (size_t)p.ld_s * 4);
    ctx->compact_smem_ok = set_smem(compact_kernel, (size_t)(p.ld_s + max_pages) * 4);
    if (!ctx->compact_smem_ok) ok = ok && set_smem(compact_kernel, (size_t)max_pages * 4);
    ctx->fused_smem = (size_t)(2 * p.ld_s + max_pages) * 4;
    ctx->fused_ok = set_smem(compress_fused_kernel, ctx->fused_smem);
    if (!ok) {
      fprintf(stderr, "scalekv_init: a slice of up to %d entries needs more shared memory than a CTA of this device has\n", p.ld_s);
      return bail(SCALEKV_ERR_UNSUPPORTED);
    }
  }
  std::string tc_err;
  if (!ctx->tc.init(cfg->dtype, p.d, ctx->pool + p.off_k, ctx->pool + p.off_v, p.n_pages, p.P, tc_err)) {
    scalekv_status s = fail(ctx, SCALEKV_ERR_CUDA, "tensor-core attend set-up failed: %s", tc_err.c_str());
    fprintf(stderr, "scalekv_init: %s\n", ctx->err.c_str());
    return bail(s);
  }
  *out = ctx;
  return SCALEKV_OK;
}

scalekv_status scalekv_reset(scalekv_ctx *ctx) {
  if (!ctx) return SCALEKV_ERR_INVALID_ARG;
  const Plan &p = ctx->plan;
  if (ctx->s_side != ctx->s_main) {
    // stream_main forks to stream_side and joins it again: everything enqueued on either stream so far
    // precedes the reset.  (Fork before join, so that the sequence is also legal while stream_main is
    // being captured into a CUDA graph.)
    CU(cudaEventRecord(ctx->ev_attend[0], ctx->s_main));
    CU(cudaStreamWaitEvent(ctx->s_side, ctx->ev_attend[0], 0));
    CU(cudaEventRecord(ctx->ev_compress[0], ctx->s_side));
    CU(cudaStreamWaitEvent(ctx->s_main, ctx->ev_compress[0], 0));
  }
  CU(cudaMemsetAsync(ctx->pool + p.off_len, 0, (size_t)p.n_layers * p.n_slices * 4, ctx->s_main));
  if (ctx->s_side != ctx->s_main) {
    // later side-stream work must not overtake the reset
    CU(cudaEventRecord(ctx->ev_attend[0], ctx->s_main));
    CU(cudaStreamWaitEvent(ctx->s_side, ctx->ev_attend[0], 0));
  }
  std::fill(ctx->next_scale.begin(), ctx->next_scale.end(), 0);
  std::fill(ctx->hist.begin(), ctx->hist.end(), 0);
  std::fill(ctx->pending.begin(), ctx->pending.end(), 0);
  std::fill(ctx->attended.begin(), ctx->attended.end(), 0);
  std::fill(ctx->in_store.begin(), ctx->in_store.end(), 1);
  std::fill(ctx->logits_of.begin(), ctx->logits_of.end(), -1);
  std::fill(ctx->ev_compress_live.begin(), ctx->ev_compress_live.end(), 0);
  for (int t = 0; t < kSets; ++t) ctx->set_owner[t] = -1;
  ctx->side_dirty = ctx->s_side != ctx->s_main;   // the side stream was sent behind the reset: a capture has to join it again
  std::fill(ctx->map_lost.begin(), ctx->map_lost.end(), 0);
  return SCALEKV_OK;
}

scalekv_status scalekv_destroy(scalekv_ctx *ctx) {
  if (!ctx) return SCALEKV_ERR_INVALID_ARG;
  cudaStreamSynchronize(ctx->s_main);
  if (ctx->s_side != ctx->s_main) cudaStreamSynchronize(ctx->s_side);
  drain_profile(ctx);
  if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
  if (ctx->s_h2d) { cudaStreamSynchronize(ctx->s_h2d); cudaStreamDestroy(ctx->s_h2d); }
  if (ctx->s_d2h) { cudaStreamSynchronize(ctx->s_d2h); cudaStreamDestroy(ctx->s_d2h); }
  for (int i = 0; i < 2; ++i) {
    if (ctx->ev_in[i]) cudaEventDestroy(ctx->ev_in[i]);
    if (ctx->ev_out[i]) cudaEventDestroy(ctx->ev_out[i]);
    if (ctx->ev_att[i]) cudaEventDestroy(ctx->ev_att[i]);
  }
  for (auto e : ctx->ev_attend) cudaEventDestroy(e);
  for (auto e : ctx->ev_compress) cudaEventDestroy(e);
  for (auto e : ctx->event_pool) cudaEventDestroy(e);
  delete ctx;
  return SCALEKV_OK;
}

scalekv_status scalekv_append(scalekv_ctx *ctx, int32_t layer, int32_t scale, scalekv_tensor K, scalekv_tensor V) {
  if (!ctx) return SCALEKV_ERR_INVALID_ARG;
  const Plan &p = ctx->plan;
  if (layer < 0 || layer >= p.n_layers) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "layer %d out of range", layer);
  if (scale < 0 || scale >= p.K) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "scale %d out of range", scale);
  if (scale != ctx->next_scale[layer])
    return fail(ctx, SCALEKV_ERR_BAD_STATE, "layer %d expects scale %d, got %d", layer, ctx->next_scale[layer], scale);
  if (!tensor_ok(K, p.esize) || !tensor_ok(V, p.esize)) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "K/V null or rows not 16-byte aligned");
  // The transient page set and the logit buffer of this layer's set (layer mod kSets) are shared with every other
  // layer of that set.  Their last user (the owner) must be through with them: a pending map of the owner whose
  // rows reach into the transient pages would be overwritten, so that order of calls is refused; otherwise
  // stream_main waits for the owner's last compress (and for this layer's own).
  const int par = layer % kSets;
  const int owner = ctx->set_owner[par];
  if (owner >= 0 && owner != layer && ctx->pending[owner] != 0) {
    const LayerPlan &op = p.layers[owner];
    if (ctx->hist[owner] + ctx->pending[owner] > op.persist_pages * p.P) {
      // the one map that nothing needs after its attend is the last scale's (no later step reads it): its
      // transient rows may go, and the layer then accepts nothing but a reset
      if (ctx->next_scale[owner] == p.K && ctx->attended[owner]) ctx->map_lost[owner] = 1;
      else
        return fail(ctx, SCALEKV_ERR_BAD_STATE,
                    "layer %d: layer %d still holds an uncompressed map in the transient pages both layers share; compress it first",
                    layer, owner);
    }
    ctx->logits_of[owner] = -1;      // its recorded window logits are about to be overwritten: score from K instead
  }
  if (ctx->s_side != ctx->s_main) {
    if (ctx->ev_compress_live[layer] && !ctx->ev_compress_joined[layer]) CU(cudaStreamWaitEvent(ctx->s_main, ctx->ev_compress[layer], 0));
    if (owner >= 0 && owner != layer && ctx->ev_compress_live[owner] && !ctx->ev_compress_joined[owner])
      CU(cudaStreamWaitEvent(ctx->s_main, ctx->ev_compress[owner], 0));
  }
  scalekv_status st = materialize(ctx, layer);
  if (st != SCALEKV_OK) return st;
  st = commit_pending(ctx, layer, ctx->s_main);
  if (st != SCALEKV_OK) return st;
  const int nk = p.n[scale];
  if (ctx->hist[layer] + nk > p.layers[layer].total_pages * p.P)
    return fail(ctx, SCALEKV_ERR_CAPACITY, "layer %d: %d + %d entries exceed the planned capacity", layer, ctx->hist[layer], nk);
  if (ctx->tc.enabled()) {
    // the tensor-core attend reads the map from K and V and copies it into the pages as it goes
    ctx->pend_k[layer] = K;
    ctx->pend_v[layer] = V;
    ctx->in_store[layer] = 0;
  } else {
    Scope sc(ctx, ctx->s_main, kAppend);
    dim3 grid((nk + 63) / 64, p.n_slices);
    append_kernel<<<grid, 256, 0, ctx->s_main>>>(layer_view(ctx, layer), tview(K), tview(V), nk, p.N[scale], p.esize);
    ctx->in_store[layer] = 1;
  }
  ctx->pending[layer] = nk;
  ctx->attended[layer] = 0;
  ctx->next_scale[layer] = scale + 1;
  ctx->set_owner[par] = layer;
  return check_launch(ctx, "append");
}

// record: whether the kernel should also record the logits of the scale's planned observation window for a compress
// that follows.  Recording costs the kernel 3-13 % (the threads that own window rows store 512 bytes per key tile and
// their tile waits for them), so it is left out where no compress can use it: after the last scale of the schedule
// (Sec. 3.3: nothing is generated after it, so the method prunes nothing there; a compress called all the same takes
// its logits from K) and in a one-call step that names no window.
// copy: whether a current map that is still in the caller's tensors is also copied into the pages while the kernel
// streams it.  A one-call step leaves the copy out when its own compress will evict (the compress then takes the
// surviving rows of the map straight from the caller's tensors: in a refiner layer 19 of 20 rows of a map would be
// written to the pages only to be dropped) and after the last scale without a compress (the rows are copied by
// whichever later call needs them, if any does).
static scalekv_status attend_impl(scalekv_ctx *ctx, int32_t layer, scalekv_tensor Q, scalekv_tensor O, float *lse, bool record,
                                  bool copy) {
  if (!ctx) return SCALEKV_ERR_INVALID_ARG;
  const Plan &p = ctx->plan;
  if (layer < 0 || layer >= p.n_layers) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "layer %d out of range", layer);
  if (ctx->pending[layer] == 0) return fail(ctx, SCALEKV_ERR_BAD_STATE, "layer %d: attend needs a preceding append", layer);
  if (!tensor_ok(Q, p.esize) || !tensor_ok(O, p.esize)) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "Q/O null or rows not 16-byte aligned");
  const int nk = ctx->pending[layer];
  LayerView lv = layer_view(ctx, layer);
  if (!ctx->tc.enabled()) {
    scalekv_status st = materialize(ctx, layer);
    if (st != SCALEKV_OK) return st;
  }
  {
    Scope sc(ctx, ctx->s_main, kAttend);
    if (ctx->tc.enabled()) {
      std::string e;
      const bool fused = !ctx->in_store[layer];
      TensorView kc, vc;
      if (fused) { kc = tview(ctx->pend_k[layer]); vc = tview(ctx->pend_v[layer]); }
      const int k = ctx->next_scale[layer] - 1;
      const std::vector<int> &win = p.windows[k];
      float *wl = (win.empty() || !record || k + 1 == p.K)
                      ? nullptr
                      : reinterpret_cast<float *>(ctx->ws + p.off_logits) + (size_t)(layer % kSets) * p.logits_elems;
      float *wlse = reinterpret_cast<float *>(ctx->ws + p.off_wlse) + (size_t)(layer % kSets) * p.n_slices * p.max_window;
      if (!ctx->tc.launch(lv, tview(Q), tview(O), lse, nk, fused ? &kc : nullptr, fused ? &vc : nullptr, fused && copy, p.N[k],
                          ctx->scale, wl, wlse, p.ld_l, win.data(), (int)win.size(), ctx->s_main, e))
        return fail(ctx, SCALEKV_ERR_CUDA, "attend launch: %s", e.c_str());
      if (copy) ctx->in_store[layer] = 1;
      ctx->logits_of[layer] = wl ? k : -1;
      ctx->logits_padded[layer] = fused ? 1 : 0;
    } else {
      dim3 grid((nk + 63) / 64, p.n_slices);
      if (ctx->dtype == SCALEKV_BF16)
        attend_simt_kernel<__nv_bfloat16, 128><<<grid, 256, (64 * 132 * 2 + 64 * 65 + 192) * 4, ctx->s_main>>>(
            lv, tview(Q), tview(O), lse, nk, ctx->scale);
      else
        attend_simt_kernel<float, 64><<<grid, 256, (64 * 68 * 2 + 64 * 65 + 192) * 4, ctx->s_main>>>(
            lv, tview(Q), tview(O), lse, nk, ctx->scale);
    }
  }
  ctx->attended[layer] = 1;
  if (ctx->s_side != ctx->s_main) CU(cudaEventRecord(ctx->ev_attend[layer], ctx->s_main));
  return check_launch(ctx, "attend");
}

scalekv_status scalekv_attend(scalekv_ctx *ctx, int32_t layer, scalekv_tensor Q, scalekv_tensor O, float *lse) {
  return attend_impl(ctx, layer, Q, O, lse, true, true);
}

scalekv_status scalekv_compress(scalekv_ctx *ctx, int32_t layer, scalekv_tensor Qw, int32_t w, const int32_t *window_pos,
                                int32_t qw_is_full_map) {
  return scalekv_compress_ex(ctx, layer, Qw, w, window_pos, qw_is_full_map, nullptr);
}

scalekv_status scalekv_compress_ex(scalekv_ctx *ctx, int32_t layer, scalekv_tensor Qw, int32_t w, const int32_t *window_pos,
                                   int32_t qw_is_full_map, const scalekv_select_opts *opts) {
  if (!ctx) return SCALEKV_ERR_INVALID_ARG;
  const Plan &p = ctx->plan;
  if (layer < 0 || layer >= p.n_layers) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "layer %d out of range", layer);
  if (ctx->pending[layer] == 0) return fail(ctx, SCALEKV_ERR_BAD_STATE, "layer %d: compress needs a preceding append", layer);
  if (ctx->map_lost[layer]) return fail(ctx, SCALEKV_ERR_BAD_STATE, "layer %d: the rows of its last map were handed to another layer after its attend", layer);
  const int policy = opts ? opts->policy : SCALEKV_SELECT_SCORE;
  const int pool = (opts && opts->pool_kernel > 1) ? opts->pool_kernel : 1;
  const int n_sink = opts ? opts->n_sink : 0;
  const bool head_shared = opts && opts->head_shared != 0 && (opts->policy == SCALEKV_SELECT_SCORE);
  if (policy != SCALEKV_SELECT_SCORE && policy != SCALEKV_SELECT_RECENT) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "unknown selection policy %d", policy);
  if (pool % 2 == 0 || pool > 63) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "pool_kernel must be odd and below 64");
  if (n_sink < 0) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "n_sink must not be negative");
  if (head_shared && p.H > 256) return fail(ctx, SCALEKV_ERR_UNSUPPORTED, "head_shared supports at most 256 heads");
  const int32_t *head_budgets = opts ? opts->head_budgets : nullptr;
  if (head_budgets && p.H > kMaxHeadBudgets) return fail(ctx, SCALEKV_ERR_UNSUPPORTED, "head_budgets supports at most %d heads", kMaxHeadBudgets);
  const bool recent = policy == SCALEKV_SELECT_RECENT;
  const int k = ctx->next_scale[layer] - 1;
  const int L = ctx->hist[layer] + ctx->pending[layer];
  WindowArg wa;
  scalekv_status st = SCALEKV_OK;
  int always_kept;       // entries outside the selection: the window, or the sinks
  if (recent) {
    // no observation window: every entry but the sinks competes on its original position
    wa.w = 0; wa.all = 0; wa.n_prev = p.N[k]; wa.n_k = p.n[k];
    for (int j = 0; j < kMaxWindow; ++j) wa.pos[j] = 0x7fffffff;
    always_kept = std::min(n_sink, p.N[k + 1]);          // positions 0 .. n_sink-1 are never evicted once appended
    {
      // the pages were sized for the table's value: sinks beyond it would be left in pages shared with other layers
      const int tab = p.budgets[(size_t)layer * p.K + k];
      const LayerPlan &lp = p.layers[layer];
      if (tab != SCALEKV_KEEP_ALL && lp.persist_pages < lp.total_pages && std::max(tab, always_kept) > lp.persist_pages * p.P)
        return fail(ctx, SCALEKV_ERR_CAPACITY, "layer %d: %d sinks exceed the persistent capacity %d planned from the budget table",
                    layer, always_kept, lp.persist_pages * p.P);
    }
  } else {
    if (!tensor_ok(Qw, p.esize)) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "Qw null or rows not 16-byte aligned");
    st = fill_window(ctx, layer, w, window_pos, wa);
    if (st != SCALEKV_OK) return st;
    always_kept = wa.w;
  }
  const int cand = L - always_kept;
  const int table = p.budgets[(size_t)layer * p.K + k];
  // SCORE: k^l counts the selected entries, the window comes on top.  RECENT: k^l is the whole cache, sinks included.
  int budget = (recent && table != SCALEKV_KEEP_ALL) ? std::max(table - always_kept, 0) : table;
  HeadBudgets hb{};
  bool hb_on = false;
  if (head_budgets) {
    // per-head budgets of this call: the same conversion as for the table's value; the call's common
    // budget becomes their maximum, which bounds the lengths the host assumes afterwards
    int lo = 0x7fffffff, hi = 0;
    for (int h = 0; h < p.H; ++h) {
      const int b = head_budgets[h];
      if (b < 0 || (table != SCALEKV_KEEP_ALL && b > table))
        return fail(ctx, SCALEKV_ERR_INVALID_ARG, "head_budgets[%d] = %d outside [0, %d]", h, b, table);
      hb.v[h] = recent ? std::max(b - always_kept, 0) : b;
      lo = std::min(lo, hb.v[h]); hi = std::max(hi, hb.v[h]);
    }
    if (head_shared && lo != hi) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "head_shared needs equal head_budgets");
    hb_on = true;
    budget = std::min(hi, cand);
    if (lo >= cand) hb_on = false, budget = SCALEKV_KEEP_ALL;      // no head evicts anything
  }
  const bool evict = budget != SCALEKV_KEEP_ALL && (budget < cand || hb_on);
  // while per-kernel timing is on, compress runs on stream_main too, so that every kernel is timed alone
  cudaStream_t s = ctx->serialize ? ctx->s_main : ctx->s_side;
  // the logits of exactly this window may already be there, recorded by attend
  bool recorded = recent || (ctx->logits_of[layer] == k && (int)p.windows[k].size() == wa.w);
  for (int j = 0; !recent && recorded && j < wa.w; ++j) recorded = p.windows[k][j] == wa.pos[j];
  const bool fused = ctx->fused_ok && !head_shared && !(opts && opts->separate_kernels);
  // A map that attend left in the caller's tensors stays there when the one-launch compress can do without the pages:
  // it needs no K (the logits are recorded) and takes the surviving rows from the tensors.  Everything else copies first.
  const bool external = !ctx->in_store[layer] && ctx->attended[layer] && evict && fused && recorded;
  const bool copy_now = !ctx->in_store[layer] && !external;
  if (!external) {
    st = materialize(ctx, layer);
    if (st != SCALEKV_OK) return st;
  }
  if (s != ctx->s_main) {
    if (!ctx->attended[layer] || copy_now) CU(cudaEventRecord(ctx->ev_attend[layer], ctx->s_main));
    CU(cudaStreamWaitEvent(s, ctx->ev_attend[layer], 0));
  }
  if (!evict) {
    st = commit_pending(ctx, layer, s);
    if (st != SCALEKV_OK) return st;
  } else {
    LayerView lv = layer_view(ctx, layer);
    float *logits = reinterpret_cast<float *>(ctx->ws + p.off_logits) + (size_t)(layer % kSets) * p.logits_elems;
    float *scores = reinterpret_cast<float *>(ctx->ws + p.off_scores);
    int *keep = reinterpret_cast<int *>(ctx->ws + p.off_keep);
    int *kept = reinterpret_cast<int *>(ctx->ws + p.off_kept);
    uint32_t *keys = reinterpret_cast<uint32_t *>(ctx->ws + p.off_keys);
    if (recent && !fused) {
      Scope sc(ctx, s, kScore);
      recent_keys_kernel<<<dim3((L + 255) / 256, p.n_slices), 256, 0, s>>>(lv, wa.n_k, n_sink, keys, p.ld_s);
    }
    if (!recorded) {
      // this writes the logit buffer of the layer's set: if another layer of that set has appended since, what
      // its attend recorded there is lost (its compress scores from K too), and its attend must be through first
      const int ow = ctx->set_owner[layer % kSets];
      if (ow >= 0 && ow != layer) {
        ctx->logits_of[ow] = -1;
        if (s != ctx->s_main && ctx->attended[ow]) CU(cudaStreamWaitEvent(s, ctx->ev_attend[ow], 0));
      }
    }
    if (!recorded) {
      Scope sc(ctx, s, kScore);
      dim3 grid((L + 63) / 64, p.n_slices);
      if (ctx->dtype == SCALEKV_BF16)
        score_logits_kernel<__nv_bfloat16, 128><<<grid, 256, 2 * 64 * 132 * 4, s>>>(lv, tview(Qw), wa, qw_is_full_map, logits,
                                                                                  p.ld_l, ctx->scale);
      else
        score_logits_kernel<float, 64><<<grid, 256, 2 * 64 * 68 * 4, s>>>(lv, tview(Qw), wa, qw_is_full_map, logits, p.ld_l,
                                                                         ctx->scale);
    }
    ctx->logits_of[layer] = -1;
    float *wlse = reinterpret_cast<float *>(ctx->ws + p.off_wlse) + (size_t)(layer % kSets) * p.n_slices * p.max_window;
    if (!recorded) {
      Scope sc(ctx, s, kScore);
      row_lse_kernel<<<p.n_slices, 1024, 0, s>>>(lv, wa, logits, p.ld_l, wlse);
    }
    // logits recorded by attend are raw products in the tile-aligned layout; the logits kernel writes base-2 logits by slot
    const float logit_scale = recorded ? ctx->scale * 1.4426950408889634f : 1.f;
    const int tile_padded = (recorded && ctx->logits_padded[layer]) ? 1 : 0;
    int *slice_budget = nullptr;
    if (hb_on) {
      slice_budget = reinterpret_cast<int *>(ctx->ws + p.off_hbud);
      Scope sc(ctx, s, kSelect);
      head_budget_kernel<<<(p.n_slices + 255) / 256, 256, 0, s>>>(hb, p.H, p.n_slices, slice_budget);
    }
    if (fused) {
      // importance, selection and pruning of a slice by one CTA, in one launch
      Scope sc(ctx, s, kCompress);
      ExternalMap ext{};
      if (external) {
        const TensorView kc = tview(ctx->pend_k[layer]), vc = tview(ctx->pend_v[layer]);
        ext.on = 1; ext.k = kc.ptr; ext.v = vc.ptr; ext.sb = kc.sb; ext.sh = kc.sh; ext.st = kc.st; ext.esize = p.esize;
        if (vc.sb != kc.sb || vc.sh != kc.sh || vc.st != kc.st) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "K and V of a map must have the same strides");
      }
      compress_fused_kernel<<<p.n_slices, 1024, ctx->fused_smem, s>>>(lv, wa, recent ? 1 : 0, n_sink, logits, wlse, p.ld_l, logit_scale,
                                                                     tile_padded, budget, slice_budget, pool, scores, p.ld_s, kept, ext);
      if (external) ctx->in_store[layer] = 1;
    } else {
      if (!recent) {
        Scope sc(ctx, s, kScore);
        score_kernel<<<dim3((L + 255) / 256, p.n_slices), 256, 0, s>>>(lv, wa, logits, wlse, p.ld_l, logit_scale, tile_padded, scores,
                                                                       keys, p.ld_s);
      }
      if (head_shared) {
        Scope sc(ctx, s, kScore);
        head_mean_kernel<<<dim3((L + 255) / 256, p.n_slices / p.H), 256, 0, s>>>(lv, wa, scores, keys, p.ld_s);
      }
      {
        Scope sc(ctx, s, kSelect);
        select_kernel<<<p.n_slices, 1024, ctx->select_smem_ok ? (size_t)p.ld_s * 4 : 0, s>>>(
            lv, wa, budget, slice_budget, keys, recent ? nullptr : scores, pool, p.ld_s, ctx->select_smem_ok ? 1 : 0, keep, kept);
      }
      {
        Scope sc(ctx, s, kCompact);
        const size_t sm = (size_t)(lv.pages_per_slice + (ctx->compact_smem_ok ? p.ld_s : 0)) * 4;
        compact_kernel<<<dim3(p.n_slices, 2, 4), 256, sm, s>>>(lv, keep, p.ld_s, ctx->compact_smem_ok ? 1 : 0, kept);
      }
    }
    ctx->scores_len = recent ? 0 : L;
    ctx->hist[layer] = budget + always_kept;
    ctx->pending[layer] = 0;
    ctx->attended[layer] = 0;
    st = check_launch(ctx, "compress");
    if (st != SCALEKV_OK) return st;
  }
  if (s != ctx->s_main) {
    CU(cudaEventRecord(ctx->ev_compress[layer], s));
    ctx->side_dirty = true;
    ctx->ev_compress_live[layer] = 1;
    ctx->ev_compress_joined[layer] = 0;
  }
  return SCALEKV_OK;
}

scalekv_status scalekv_step_host(scalekv_ctx *ctx, int32_t layer, int32_t scale, const void *Q_host, const void *K_host,
                                 const void *V_host, void *O_host, void *staging, size_t staging_bytes, int32_t w,
                                 const int32_t *window_pos) {
  if (!ctx) return SCALEKV_ERR_INVALID_ARG;
  const Plan &p = ctx->plan;
  if (scale < 0 || scale >= p.K) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "scale %d out of range", scale);
  if (!Q_host || !K_host || !V_host || !O_host || !staging) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "null buffer");
  const int nk = p.n[scale];
  const size_t bytes = (size_t)p.n_slices * nk * p.d * p.esize;
  if (staging_bytes < 8 * bytes) return fail(ctx, SCALEKV_ERR_CAPACITY, "staging needs %zu bytes", 8 * bytes);
  if (!ctx->s_h2d) {
    // first use: two copy streams of the library's own (input and output copies run in both directions
    // at once and under the kernels of neighbouring steps) and the events that chain them
    CU(cudaStreamCreateWithFlags(&ctx->s_h2d, cudaStreamNonBlocking));
    CU(cudaStreamCreateWithFlags(&ctx->s_d2h, cudaStreamNonBlocking));
    for (int i = 0; i < 2; ++i) {
      CU(cudaEventCreateWithFlags(&ctx->ev_in[i], cudaEventDisableTiming));
      CU(cudaEventCreateWithFlags(&ctx->ev_out[i], cudaEventDisableTiming));
      CU(cudaEventCreateWithFlags(&ctx->ev_att[i], cudaEventDisableTiming));
    }
  }
  // consecutive steps alternate between the two halves of the staging area
  const int set = (int)(ctx->host_steps++ & 1);
  char *dq = static_cast<char *>(staging) + (size_t)set * 4 * bytes, *dk = dq + bytes, *dv = dk + bytes, *dout = dv + bytes;
  if (ctx->set_layer[set] >= 0) {
    // the half's previous user must be through: its output copied out, its compress (which may read Q) done
    CU(cudaStreamWaitEvent(ctx->s_h2d, ctx->ev_out[set], 0));
    const int pl = ctx->set_layer[set];
    if (ctx->ev_compress_live[pl]) CU(cudaStreamWaitEvent(ctx->s_h2d, ctx->ev_compress[pl], 0));
    else CU(cudaStreamWaitEvent(ctx->s_h2d, ctx->ev_att[set], 0));
  }
  CU(cudaMemcpyAsync(dk, K_host, bytes, cudaMemcpyHostToDevice, ctx->s_h2d));
  CU(cudaMemcpyAsync(dv, V_host, bytes, cudaMemcpyHostToDevice, ctx->s_h2d));
  CU(cudaMemcpyAsync(dq, Q_host, bytes, cudaMemcpyHostToDevice, ctx->s_h2d));
  CU(cudaEventRecord(ctx->ev_in[set], ctx->s_h2d));
  CU(cudaStreamWaitEvent(ctx->s_main, ctx->ev_in[set], 0));
  auto dense = [&](const void *ptr) {
    scalekv_tensor t; t.ptr = ptr; t.stride_t = p.d; t.stride_h = (int64_t)nk * p.d; t.stride_b = (int64_t)p.H * nk * p.d;
    return t;
  };
  scalekv_status st = scalekv_append(ctx, layer, scale, dense(dk), dense(dv));
  if (st != SCALEKV_OK) return st;
  st = scalekv_attend(ctx, layer, dense(dq), dense(dout), nullptr);
  if (st != SCALEKV_OK) return st;
  CU(cudaEventRecord(ctx->ev_att[set], ctx->s_main));
  CU(cudaStreamWaitEvent(ctx->s_d2h, ctx->ev_att[set], 0));
  CU(cudaMemcpyAsync(O_host, dout, bytes, cudaMemcpyDeviceToHost, ctx->s_d2h));
  CU(cudaEventRecord(ctx->ev_out[set], ctx->s_d2h));
  ctx->set_layer[set] = layer;
  if (w > 0) {
    st = scalekv_compress(ctx, layer, dense(dq), w, window_pos, 1);
    if (st != SCALEKV_OK) return st;
  } else if (w < 0) {
    st = scalekv_compress(ctx, layer, dense(dq), 0, nullptr, 1);
    if (st != SCALEKV_OK) return st;
  }
  return SCALEKV_OK;
}

// Whether the attend of a one-call step copies the current map into the pages (see attend_impl).  It does not when
// the step's own compress will evict - the test scalekv_compress_ex makes - and will find what it needs without K in
// the pages (the logits of exactly its window recorded, or a positional rule), so that it can take the map's
// surviving rows from K and V itself; nor after the last scale without a compress, when nothing may ever need the rows.
// A wrong guess costs a copy kernel, never a result.
static bool step_copies(const scalekv_ctx *ctx, int layer, int scale, bool compress, int w, const int32_t *window_pos,
                        const scalekv_select_opts *opts) {
  if (!ctx || !ctx->tc.enabled() || layer < 0 || layer >= ctx->plan.n_layers || scale < 0 || scale >= ctx->plan.K) return true;
  const Plan &p = ctx->plan;
  if (!compress) return scale + 1 != p.K;
  if (!ctx->fused_ok || (opts && (opts->head_shared || opts->separate_kernels || opts->head_budgets))) return true;
  const int table = p.budgets[(size_t)layer * p.K + scale];
  if (table == SCALEKV_KEEP_ALL) return true;
  const int L = ctx->hist[layer] + p.n[scale];
  if (opts && opts->policy == SCALEKV_SELECT_RECENT) {
    const int sinks = std::min(std::max(opts->n_sink, 0), p.N[scale + 1]);
    return !(std::max(table - sinks, 0) < L - sinks);
  }
  if (w <= 0) return true;
  bool planned = scale + 1 != p.K && window_pos && (int)p.windows[scale].size() == w;
  for (int j = 0; planned && j < w; ++j) planned = p.windows[scale][j] == window_pos[j];
  return !(planned && table < L - w);
}

scalekv_status scalekv_step(scalekv_ctx *ctx, int32_t layer, int32_t scale, scalekv_tensor Q, scalekv_tensor K, scalekv_tensor V,
                            scalekv_tensor O, float *lse, int32_t w, const int32_t *window_pos) {
  scalekv_status st = scalekv_append(ctx, layer, scale, K, V);
  if (st != SCALEKV_OK) return st;
  st = attend_impl(ctx, layer, Q, O, lse, w > 0, step_copies(ctx, layer, scale, w != 0, w, window_pos, nullptr));
  if (st != SCALEKV_OK) return st;
  if (w > 0) return scalekv_compress(ctx, layer, Q, w, window_pos, 1);
  if (w < 0) return scalekv_compress(ctx, layer, Q, 0, nullptr, 1);
  return SCALEKV_OK;
}

scalekv_status scalekv_step_ex(scalekv_ctx *ctx, int32_t layer, int32_t scale, scalekv_tensor Q, scalekv_tensor K, scalekv_tensor V,
                               scalekv_tensor O, float *lse, int32_t compress, int32_t w, const int32_t *window_pos,
                               const scalekv_select_opts *opts) {
  scalekv_status st = scalekv_append(ctx, layer, scale, K, V);
  if (st != SCALEKV_OK) return st;
  const bool score = !opts || opts->policy == SCALEKV_SELECT_SCORE;
  st = attend_impl(ctx, layer, Q, O, lse, compress != 0 && score && w > 0,
                   step_copies(ctx, layer, scale, compress != 0, w, window_pos, opts));
  if (st != SCALEKV_OK) return st;
  if (!compress) return SCALEKV_OK;
  return scalekv_compress_ex(ctx, layer, Q, w, window_pos, 1, opts);
}

scalekv_status scalekv_layer_stats(scalekv_ctx *ctx, int32_t layer, scalekv_tensor Q, int32_t topk_prime,
                                   int32_t query_stride, double *car, double *htk) {
  return scalekv_layer_stats_ex(ctx, layer, Q, topk_prime, query_stride, car, htk, nullptr, nullptr, nullptr);
}

scalekv_status scalekv_layer_stats_ex(scalekv_ctx *ctx, int32_t layer, scalekv_tensor Q, int32_t topk_prime,
                                      int32_t query_stride, double *car, double *htk, double *car_slices,
                                      double *htk_slices, double *nca_slices) {
  if (!ctx || !car || !htk) return SCALEKV_ERR_INVALID_ARG;
  const Plan &p = ctx->plan;
  if (layer < 0 || layer >= p.n_layers) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "layer %d out of range", layer);
  if (ctx->pending[layer] == 0) return fail(ctx, SCALEKV_ERR_BAD_STATE, "layer %d: layer_stats needs a preceding append", layer);
  if (ctx->map_lost[layer]) return fail(ctx, SCALEKV_ERR_BAD_STATE, "layer %d: the rows of its last map were handed to another layer after its attend", layer);
  if (topk_prime < 0 || topk_prime > 64 || query_stride < 1) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "topk_prime in [0,64], stride >= 1");
  if (!tensor_ok(Q, p.esize)) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "Q null or rows not 16-byte aligned");
  scalekv_status st0 = materialize(ctx, layer);
  if (st0 != SCALEKV_OK) return st0;
  const int nk = ctx->pending[layer];
  const int k = ctx->next_scale[layer] - 1;
  const int rows = (nk + query_stride - 1) / query_stride;
  double *acc = reinterpret_cast<double *>(ctx->ws + p.off_acc);
  const size_t acc_bytes = 16 + (size_t)p.n_slices * 16;
  CU(cudaMemsetAsync(acc, 0, acc_bytes, ctx->s_main));
  // few slices and few sampled rows leave most SMs idle: split every slice's keys over enough CTAs to fill them
  const int row_blocks = (rows + 63) / 64;
  const int tiles = (ctx->hist[layer] + nk + 63) / 64;
  int n_split = 1;
  while (n_split < 16 && row_blocks * p.n_slices * n_split * 2 <= kStatsMaxCtas && n_split * 2 <= tiles) n_split *= 2;
  float *partial = reinterpret_cast<float *>(ctx->ws + p.off_stats);
  {
    Scope sc(ctx, ctx->s_main, kOther);
    dim3 grid(row_blocks, p.n_slices, n_split);
    if (ctx->dtype == SCALEKV_BF16)
      layer_stats_kernel<__nv_bfloat16, 128><<<grid, 256, layer_stats_smem_bytes<128>(topk_prime), ctx->s_main>>>(
          layer_view(ctx, layer), tview(Q), nk, p.N[k], query_stride, rows, topk_prime, ctx->scale, acc, partial);
    else
      layer_stats_kernel<float, 64><<<grid, 256, layer_stats_smem_bytes<64>(topk_prime), ctx->s_main>>>(
          layer_view(ctx, layer), tview(Q), nk, p.N[k], query_stride, rows, topk_prime, ctx->scale, acc, partial);
  }
  if (n_split > 1) {
    Scope sc(ctx, ctx->s_main, kOther);
    layer_stats_merge_kernel<<<dim3(row_blocks, p.n_slices), 64, 0, ctx->s_main>>>(partial, n_split, rows, topk_prime, acc);
  }
  scalekv_status st = check_launch(ctx, "layer_stats");
  if (st != SCALEKV_OK) return st;
  std::vector<double> host(2 + 2 * (size_t)p.n_slices);
  std::vector<int> len(p.n_slices);
  CU(cudaMemcpyAsync(host.data(), acc, acc_bytes, cudaMemcpyDeviceToHost, ctx->s_main));
  CU(cudaMemcpyAsync(len.data(), ctx->pool + p.off_len + (size_t)layer * p.n_slices * 4, (size_t)p.n_slices * 4,
                     cudaMemcpyDeviceToHost, ctx->s_main));
  CU(cudaStreamSynchronize(ctx->s_main));
  const double cnt = (double)rows * p.n_slices;
  *car = host[0] / cnt;
  *htk = host[1] / cnt;
  for (int s = 0; s < p.n_slices; ++s) {
    const double c_s = host[2 + 2 * s] / rows, t_s = host[3 + 2 * s] / rows;
    if (car_slices) car_slices[s] = c_s;
    if (htk_slices) htk_slices[s] = t_s;
    // the stored length does not count the map just appended until a compress commits it
    if (nca_slices) nca_slices[s] = c_s * (double)(len[s] + nk) / (double)nk;
  }
  return SCALEKV_OK;
}

scalekv_status scalekv_window_centroids(int32_t h, int32_t w, int32_t n_patches, int32_t *pos, int32_t *count) {
  if (h < 1 || w < 1 || n_patches < 1 || !pos || !count) return SCALEKV_ERR_INVALID_ARG;
  const std::vector<int> out = centroid_window(h, w, n_patches);
  for (size_t i = 0; i < out.size(); ++i) pos[i] = out[i];
  *count = (int)out.size();
  return SCALEKV_OK;
}

scalekv_status scalekv_assign_roles(const double *asi, int32_t L, int32_t K, int32_t n_drafters, int32_t mode, double eps,
                                    uint8_t *is_drafter) {
  if (!asi || !is_drafter || L < 1 || K < 1 || n_drafters < 0) return SCALEKV_ERR_INVALID_ARG;
  std::vector<double> z((size_t)L * K, 0.0);
  for (int k = 0; k < K; ++k) {
    double mu = 0; for (int l = 0; l < L; ++l) mu += asi[(size_t)l * K + k];
    mu /= L;
    double var = 0; for (int l = 0; l < L; ++l) { double dlt = asi[(size_t)l * K + k] - mu; var += dlt * dlt; }
    const double sd = std::sqrt(var / L);
    for (int l = 0; l < L; ++l) z[(size_t)l * K + k] = (asi[(size_t)l * K + k] - mu) / (sd + eps);
  }
  std::memset(is_drafter, 0, (size_t)L * K);
  struct Cell { double z; int k, l; };
  auto less = [](const Cell &a, const Cell &b) { return a.z != b.z ? a.z < b.z : (a.k != b.k ? a.k < b.k : a.l < b.l); };
  if (mode == 0) {
    std::vector<Cell> cells;
    for (int k = 1; k < K - 1; ++k) for (int l = 0; l < L; ++l) cells.push_back({z[(size_t)l * K + k], k, l});
    std::sort(cells.begin(), cells.end(), less);
    for (int i = 0; i < n_drafters && i < (int)cells.size(); ++i) is_drafter[(size_t)cells[i].l * K + cells[i].k] = 1;
  } else {
    for (int k = 1; k < K - 1; ++k) {
      std::vector<Cell> cells;
      for (int l = 0; l < L; ++l) cells.push_back({z[(size_t)l * K + k], k, l});
      std::sort(cells.begin(), cells.end(), less);
      for (int i = 0; i < n_drafters && i < L; ++i) is_drafter[(size_t)cells[i].l * K + k] = 1;
    }
  }
  return SCALEKV_OK;
}

scalekv_status scalekv_make_budgets(const uint8_t *is_drafter, int32_t L, int32_t K, double b_uniform, double b_r0, double delta,
                                    int32_t *budgets_out) {
  if (!is_drafter || !budgets_out || L < 1 || K < 1) return SCALEKV_ERR_INVALID_ARG;
  for (int k = 0; k < K; ++k) {
    int nd = 0; for (int l = 0; l < L; ++l) nd += is_drafter[(size_t)l * K + k] ? 1 : 0;
    const int nr = L - nd;
    const double br = std::max(b_r0 - delta * (k + 1), 0.0);
    if (nd == 0) {
      for (int l = 0; l < L; ++l) budgets_out[(size_t)l * K + k] = (int32_t)std::floor(b_uniform + 0.5);
      continue;
    }
    const double bd = (b_uniform * L - nr * br) / nd;
    for (int l = 0; l < L; ++l)
      budgets_out[(size_t)l * K + k] = (int32_t)std::floor((is_drafter[(size_t)l * K + k] ? bd : br) + 0.5);
  }
  return SCALEKV_OK;
}

scalekv_status scalekv_window_last(int32_t h, int32_t w, int32_t n_obs, int32_t *pos, int32_t *count) {
  if (h < 1 || w < 1 || n_obs < 1 || !pos || !count) return SCALEKV_ERR_INVALID_ARG;
  const long long n = (long long)h * w;
  const int m = (int)std::min<long long>(n_obs, n);
  for (int i = 0; i < m; ++i) pos[i] = (int32_t)(n - m + i);
  *count = m;
  return SCALEKV_OK;
}

scalekv_status scalekv_policy_budgets(int32_t shape, int32_t L, int32_t K, double b_mean, double beta, int32_t *budgets_out) {
  if (!budgets_out || L < 1 || K < 1 || !(b_mean >= 0.0)) return SCALEKV_ERR_INVALID_ARG;
  if (shape != SCALEKV_BUDGETS_UNIFORM && shape != SCALEKV_BUDGETS_PYRAMID) return SCALEKV_ERR_INVALID_ARG;
  if (shape == SCALEKV_BUDGETS_PYRAMID && !(beta >= 1.0)) return SCALEKV_ERR_INVALID_ARG;
  for (int l = 0; l < L; ++l) {
    double b = b_mean;
    if (shape == SCALEKV_BUDGETS_PYRAMID && L > 1) {
      const double b_min = b_mean / beta, b_max = 2.0 * b_mean - b_min;
      b = b_max - (b_max - b_min) * l / (L - 1);
    }
    const int32_t v = (int32_t)std::floor(b + 0.5);
    for (int k = 0; k < K; ++k) budgets_out[(size_t)l * K + k] = v;
  }
  return SCALEKV_OK;
}

scalekv_status scalekv_budget_tokens(double fraction, const int32_t *scale_h, const int32_t *scale_w, int32_t n_scales,
                                     int32_t *tokens) {
  if (!scale_h || !scale_w || !tokens || n_scales < 1 || !(fraction >= 0.0)) return SCALEKV_ERR_INVALID_ARG;
  long long t_c = 0;
  for (int k = 0; k + 1 < n_scales; ++k) {
    if (scale_h[k] < 1 || scale_w[k] < 1) return SCALEKV_ERR_INVALID_ARG;
    t_c += (long long)scale_h[k] * scale_w[k];
  }
  const double v = std::floor(fraction * (double)t_c + 0.5 + 1e-9);   // a decimal fraction that lands on .5 rounds up
  if (v > 2147483647.0) return SCALEKV_ERR_INVALID_ARG;
  *tokens = (int32_t)v;
  return SCALEKV_OK;
}

scalekv_status scalekv_selftest_wait(scalekv_ctx *ctx, int32_t limit_ms, int32_t *gave_up, int32_t *seen_by_peer) {
  if (!ctx || !gave_up || !seen_by_peer) return SCALEKV_ERR_INVALID_ARG;
  if (limit_ms < 1 || limit_ms > 1000) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "limit_ms must lie in [1, 1000]");
  const Plan &p = ctx->plan;
  int *out = reinterpret_cast<int *>(ctx->ws + p.off_acc);
  CU(cudaMemsetAsync(out, 0, 8, ctx->s_main));
  {
    Scope sc(ctx, ctx->s_main, kOther);
    tc::wait_probe_kernel<<<1, 64, 0, ctx->s_main>>>(reinterpret_cast<int *>(ctx->pool + p.off_status),
                                                     (unsigned long long)limit_ms * 1000000ull, out);
  }
  scalekv_status st = check_launch(ctx, "wait probe");
  if (st != SCALEKV_OK) return st;
  int host[2] = {0, 0};
  CU(cudaMemcpyAsync(host, out, 8, cudaMemcpyDeviceToHost, ctx->s_main));
  CU(cudaStreamSynchronize(ctx->s_main));
  *gave_up = host[0];
  *seen_by_peer = host[1];
  return SCALEKV_OK;
}

scalekv_status scalekv_join(scalekv_ctx *ctx) {
  if (!ctx) return SCALEKV_ERR_INVALID_ARG;
  if (ctx->s_side != ctx->s_main && ctx->side_dirty) {   // (nothing enqueued there since the last join: nothing to wait for)
    CU(cudaEventRecord(ctx->ev_join, ctx->s_side));
    CU(cudaStreamWaitEvent(ctx->s_main, ctx->ev_join, 0));
    // stream_main is now behind every compress enqueued so far: later appends need not wait for them again
    // (which also lets the next scale-step be captured into a graph of its own)
    std::fill(ctx->ev_compress_joined.begin(), ctx->ev_compress_joined.end(), 1);
    ctx->side_dirty = false;
  }
  return SCALEKV_OK;
}

scalekv_status scalekv_sync(scalekv_ctx *ctx) {
  if (!ctx) return SCALEKV_ERR_INVALID_ARG;
  CU(cudaStreamSynchronize(ctx->s_main));
  if (ctx->s_side != ctx->s_main) CU(cudaStreamSynchronize(ctx->s_side));
  if (ctx->s_h2d) CU(cudaStreamSynchronize(ctx->s_h2d));
  if (ctx->s_d2h) CU(cudaStreamSynchronize(ctx->s_d2h));
  int status = 0;
  CU(cudaMemcpy(&status, ctx->pool + ctx->plan.off_status, 4, cudaMemcpyDeviceToHost));
  if (status == kDevTimeout) return fail(ctx, SCALEKV_ERR_TIMEOUT, "a bounded device-side wait gave up");
  if (status != 0) return fail(ctx, SCALEKV_ERR_DEVICE_CHECK, "device-side check failed (code %d)", status);
  return SCALEKV_OK;
}

scalekv_status scalekv_lengths(scalekv_ctx *ctx, int32_t layer, int32_t *len_host) {
  if (!ctx || !len_host) return SCALEKV_ERR_INVALID_ARG;
  const Plan &p = ctx->plan;
  if (layer < 0 || layer >= p.n_layers) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "layer %d out of range", layer);
  scalekv_status st = scalekv_sync(ctx);
  if (st != SCALEKV_OK) return st;
  CU(cudaMemcpy(len_host, ctx->pool + p.off_len + (size_t)layer * p.n_slices * 4, (size_t)p.n_slices * 4, cudaMemcpyDeviceToHost));
  for (int s = 0; s < p.n_slices; ++s) len_host[s] += ctx->pending[layer];
  return SCALEKV_OK;
}

scalekv_status scalekv_export_slice(scalekv_ctx *ctx, int32_t layer, int32_t b, int32_t h, int32_t *pos_host, void *K_host,
                                    void *V_host, int32_t cap, int32_t *len) {
  if (!ctx || !len) return SCALEKV_ERR_INVALID_ARG;
  const Plan &p = ctx->plan;
  if (layer < 0 || layer >= p.n_layers || b < 0 || b >= p.B || h < 0 || h >= p.H)
    return fail(ctx, SCALEKV_ERR_INVALID_ARG, "slice index out of range");
  scalekv_status st = materialize(ctx, layer);
  if (st != SCALEKV_OK) return st;
  st = scalekv_sync(ctx);
  if (st != SCALEKV_OK) return st;
  const int slice = b * p.H + h;
  int hist = 0;
  CU(cudaMemcpy(&hist, ctx->pool + p.off_len + ((size_t)layer * p.n_slices + slice) * 4, 4, cudaMemcpyDeviceToHost));
  const int L = hist + (ctx->map_lost[layer] ? 0 : ctx->pending[layer]);   // a given-up last map is not exported
  *len = L;
  if (L > cap) return fail(ctx, SCALEKV_ERR_CAPACITY, "slice holds %d entries, cap is %d", L, cap);
  const LayerPlan &lp = p.layers[layer];
  const size_t row_bytes = (size_t)p.d * p.esize;
  for (int s0 = 0; s0 < L; s0 += p.P) {
    const int cnt = std::min(p.P, L - s0);
    const size_t page = (size_t)ctx->page_table_host[lp.page_table_off + (size_t)slice * lp.total_pages + s0 / p.P];
    if (pos_host) CU(cudaMemcpy(pos_host + s0, ctx->pool + p.off_pos + page * p.P * 4, (size_t)cnt * 4, cudaMemcpyDeviceToHost));
    if (K_host) CU(cudaMemcpy(static_cast<char *>(K_host) + s0 * row_bytes, ctx->pool + p.off_k + page * p.P * row_bytes, cnt * row_bytes, cudaMemcpyDeviceToHost));
    if (V_host) CU(cudaMemcpy(static_cast<char *>(V_host) + s0 * row_bytes, ctx->pool + p.off_v + page * p.P * row_bytes, cnt * row_bytes, cudaMemcpyDeviceToHost));
  }
  return SCALEKV_OK;
}

scalekv_status scalekv_export_scores(scalekv_ctx *ctx, int32_t b, int32_t h, float *s_host, int32_t cap, int32_t *len) {
  if (!ctx || !s_host || !len) return SCALEKV_ERR_INVALID_ARG;
  const Plan &p = ctx->plan;
  if (b < 0 || b >= p.B || h < 0 || h >= p.H) return fail(ctx, SCALEKV_ERR_INVALID_ARG, "slice index out of range");
  scalekv_status st = scalekv_sync(ctx);
  if (st != SCALEKV_OK) return st;
  *len = ctx->scores_len;
  if (ctx->scores_len > cap) return fail(ctx, SCALEKV_ERR_CAPACITY, "scores hold %d entries, cap is %d", ctx->scores_len, cap);
  CU(cudaMemcpy(s_host, ctx->ws + p.off_scores + (size_t)(b * p.H + h) * p.ld_s * 4, (size_t)ctx->scores_len * 4, cudaMemcpyDeviceToHost));
  return SCALEKV_OK;
}

scalekv_status scalekv_launch_count(scalekv_ctx *ctx, int64_t *count) {
  if (!ctx || !count) return SCALEKV_ERR_INVALID_ARG;
  *count = ctx->launches;
  return SCALEKV_OK;
}

scalekv_status scalekv_profile_enable(scalekv_ctx *ctx, int32_t on) {
  if (!ctx) return SCALEKV_ERR_INVALID_ARG;
  scalekv_status st = scalekv_sync(ctx);
  if (st != SCALEKV_OK) return st;
  drain_profile(ctx);
  if (on) for (int i = 0; i < kNumClasses; ++i) { ctx->prof_ms[i] = 0; ctx->prof_n[i] = 0; }
  ctx->profile = on != 0;
  ctx->serialize = on == 2;
  return SCALEKV_OK;
}

scalekv_status scalekv_profile_read(scalekv_ctx *ctx, int32_t which, double *ms_total, int64_t *launches) {
  if (!ctx || which < 0 || which >= kNumClasses || !ms_total || !launches) return SCALEKV_ERR_INVALID_ARG;
  scalekv_status st = scalekv_sync(ctx);
  if (st != SCALEKV_OK) return st;
  drain_profile(ctx);
  *ms_total = ctx->prof_ms[which];
  *launches = ctx->prof_n[which];
  return SCALEKV_OK;
}

const char *scalekv_error_string(scalekv_ctx *ctx) { return ctx ? ctx->err.c_str() : "null context"; }

}  // extern "C"
