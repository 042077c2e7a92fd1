// C entry points: argument checks, workspace carving, launches, measurement hooks.
#include <new>
#include <vector>
#include <cstring>
#include "sdms_internal.h"

using namespace sdms;

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Layout {
  size_t tok, pq, len, rec, status, index, q_fp, q_mode, q_reserved, q_off, q_cursor, match_cursor, g_nscan, g_trim, matches;
  size_t w_ctl, w_desc, w_pred, w_edge, w_tab, w_key, w_item, b_ent, b_ctl, bp_todo;
  bool wide_on;
  uint64_t w_slots;
  size_t x_draft_tok, x_draft_len, x_node_tok, x_node_S, x_node_cnt, x_node_count, x_edge_dst, x_edge_S, x_edge_cnt, x_out_degree;
  size_t total;
  uint32_t table_cap;
  int64_t match_cap;
};

int check_config(const sdms_config* c) {
  if (!c || c->struct_size != sizeof(sdms_config)) return SDMS_ERR_INVALID_ARG;
  if (c->num_groups < 1 || c->paths_per_group < 1 || c->paths_per_group > SDMS_MAX_PATHS_PER_GROUP)
    return SDMS_ERR_INVALID_ARG;
  if (c->capacity < 2 || c->vocab < 1 || c->vocab > (1 << 26)) return SDMS_ERR_INVALID_ARG;
  if (c->k_max < 1 || c->k_max > SDMS_MAX_K) return SDMS_ERR_INVALID_ARG;
  if (c->index_max_n < 0 || c->index_max_n > c->k_max || c->reserved1 != 0) return SDMS_ERR_INVALID_ARG;
  if (c->max_draft_len < 1 || c->max_draft_len > SDMS_MAX_DRAFT) return SDMS_ERR_INVALID_ARG;
  if (c->max_append < 1 || c->max_append > c->max_draft_len + 1) return SDMS_ERR_INVALID_ARG;
  if (c->dag_nodes_per_layer < 0 || c->dag_nodes_per_layer > SDMS_MAX_DAG_NODES) return SDMS_ERR_INVALID_ARG;
  if (c->dag_nodes_per_layer > 0 && (c->dag_edges_per_node < 1 || c->dag_edges_per_node > SDMS_MAX_DAG_EDGES))
    return SDMS_ERR_INVALID_ARG;
  if (c->search_mode < 0 || c->search_mode > 2) return SDMS_ERR_INVALID_ARG;
  if (!(c->alpha >= 0.0f && c->alpha <= 1.0f)) return SDMS_ERR_INVALID_ARG;
  if (c->match_capacity < 0 || c->match_capacity > 0x7fffffffLL) return SDMS_ERR_INVALID_ARG;
  const int64_t P = (int64_t)c->num_groups * c->paths_per_group;
  if (P * c->capacity > 0x7fffffffLL) return SDMS_ERR_INVALID_ARG;       // positions are int32
  if (c->epsilon < 0 || c->epsilon > 1 || c->pool_mode < 0 || c->pool_mode > 2) return SDMS_ERR_INVALID_ARG;
  if (c->search_mode == 2 && c->pool_mode != 0) return SDMS_ERR_INVALID_ARG;     // the best path is a path of the DAG
  if (c->max_matches_per_path < 0 || c->max_beams < 0 || c->max_beams > SDMS_MAX_BEAMS) return SDMS_ERR_INVALID_ARG;
  if (c->max_beams > 0 && c->pool_mode != 0) return SDMS_ERR_INVALID_ARG;        // beams are paths of the DAG
  if (c->wide_table_bytes < -1 || c->wide_table_bytes > (40LL << 31)) return SDMS_ERR_INVALID_ARG;   // slots are numbered in 32 bits
  return SDMS_OK;
}

Layout make_layout(const sdms_config* c) {
  Layout l;
  const size_t P = (size_t)c->num_groups * c->paths_per_group;
  const size_t L = c->capacity, D = c->max_draft_len, B = c->dag_nodes_per_layer, Ke = c->dag_edges_per_node;
  // twice as many buckets as positions a prompt can hold: load factor <= 1/2
  uint32_t cap = 64;
  while ((size_t)cap < 2 * (size_t)c->paths_per_group * L) cap <<= 1;
  l.table_cap = cap;
  int64_t mc = c->match_capacity;
  if (mc == 0) {
    const int64_t worst = (int64_t)P * c->paths_per_group * (int64_t)L;   // every position matches every query
    mc = worst < (1LL << 26) ? worst : (1LL << 26);
  }
  l.match_cap = mc;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes); return at; };
  l.tok = take((P * L + SDMS_MAX_DRAFT + 8) * 4);
  l.pq = take((P * L + SDMS_MAX_DRAFT + 8) * 4);
  l.len = take(P * 4);
  l.rec = take(P * kRecWords * 4);
  l.status = take(4);
  l.index = take((size_t)c->num_groups * (c->index_max_n ? c->index_max_n : c->k_max) * cap * kBucketWords * 4);
  l.q_fp = take(P * 4); l.q_mode = take(P * 4); l.q_reserved = take(P * 4);
  l.q_off = take(P * 4); l.q_cursor = take(P * 4);
  l.match_cursor = take(8);
  l.g_nscan = take((size_t)c->num_groups * 4);
  l.g_trim = take((size_t)c->num_groups * 4);
  l.matches = take((size_t)mc * 4);
  l.x_draft_tok = take(P * D * 4); l.x_draft_len = take(P * 4);
  l.x_node_tok = take(P * D * B * 4); l.x_node_S = take(P * D * B * 8); l.x_node_cnt = take(P * D * B * 4);
  l.x_node_count = take(P * D * 4);
  l.x_edge_dst = take(P * D * B * Ke * 4); l.x_edge_S = take(P * D * B * Ke * 8);
  l.x_edge_cnt = take(P * D * B * Ke * 4); l.x_out_degree = take(P * D * B * 4);
  // node tables in global memory: the device-wide aggregation of large prompts and the beams.  A slot:
  // 32 bytes of sums, 4 of key, 4 per (match, layer) item, 16 per kept continuation
  const int64_t group_tokens = (int64_t)c->paths_per_group * c->capacity;
  const bool fused = group_tokens <= kFusedMaxTokens && (int64_t)P * group_tokens <= mc;
  const int64_t stride = c->max_beams > 0 ? c->max_beams : (c->search_mode == 2 ? 1 : 0);   // continuations kept per node
  const int64_t slot_bytes = 40 + 16 * stride;
  l.wide_on = !fused && c->wide_table_bytes >= 0;
  int64_t wide = c->wide_table_bytes;
  if (wide == 0) {
    wide = slot_bytes * 5 * (int64_t)D * (int64_t)c->paths_per_group * (int64_t)(P * L);   // room for every position matching every query
    if (wide > (320LL << 20)) wide = 320LL << 20;
  }
  l.w_slots = (l.wide_on || (stride > 0 && wide > 0)) ? (uint64_t)wide / slot_bytes : 0;
  l.w_ctl = take((size_t)kWideCtlWords * 8);
  l.b_ctl = take(16);
  l.bp_todo = take(P * 4);
  l.w_desc = take(l.wide_on ? (size_t)kMaxWide * 16 : 0);
  l.w_pred = take(l.wide_on ? (size_t)kMaxWide * SDMS_MAX_DRAFT * sizeof(WidePred) : 0);
  l.w_edge = take(l.wide_on ? (size_t)kMaxWide * SDMS_MAX_DRAFT * 8 : 0);
  l.w_tab = take((size_t)l.w_slots * sizeof(WideSlot));
  l.w_key = take((size_t)l.w_slots * 4);
  l.w_item = take((size_t)l.w_slots * 4);
  l.b_ent = take((size_t)l.w_slots * 16 * stride);
  l.total = o;
  return l;
}

// Small prompts: every query path gets a private slice of N*L match slots and one CTA does the whole build.
bool fits_fused(const sdms_config* c, const Layout& l) {
  const int64_t group_tokens = (int64_t)c->paths_per_group * c->capacity;
  return group_tokens <= kFusedMaxTokens &&
         (int64_t)c->num_groups * c->paths_per_group * group_tokens <= l.match_cap;
}

// Full check: field ranges, then the layout.
int check_all(const sdms_config* c, Layout* out) {
  const int rc = check_config(c);
  if (rc != SDMS_OK) return rc;
  *out = make_layout(c);
  return SDMS_OK;
}

struct EventPair { cudaEvent_t a, b; int kernel; };

}  // namespace

struct sdms_ctx {
  sdms_config cfg;
  Layout lay;
  Dev dev;
  unsigned char* ws;
  uint64_t launches;
  bool profiling;
  bool built;
  bool step_fits;                                // sdms_step runs as one cluster launch
  int32_t* x_draft_tok; int32_t* x_draft_len;   // where the export pass leaves the drafts it recomputes
  std::vector<EventPair> pending;
  std::vector<EventPair> pool;
  float prof_ms[SDMS_NUM_KERNELS];
  uint64_t prof_n[SDMS_NUM_KERNELS];
};

namespace {

constexpr size_t kMaxPendingEvents = 8192;

// Adds the `count` oldest recorded event pairs to the per-kernel totals (waiting for them) and hands
// their events back to the pool.
int drain_pending(sdms_ctx* ctx, size_t count) {
  count = count < ctx->pending.size() ? count : ctx->pending.size();
  for (size_t x = 0; x < count; ++x) {
    EventPair& e = ctx->pending[x];
    float t = 0.f;
    if (cudaEventSynchronize(e.b) != cudaSuccess || cudaEventElapsedTime(&t, e.a, e.b) != cudaSuccess)
      return SDMS_ERR_CUDA;
    ctx->prof_ms[e.kernel] += t;
    ctx->prof_n[e.kernel] += 1;
    ctx->pool.push_back(e);
  }
  ctx->pending.erase(ctx->pending.begin(), ctx->pending.begin() + count);
  return SDMS_OK;
}

// A best-path build marks the paths with more matches than its shared-memory search takes; this launch
// searches them over node tables in the workspace's table area and replaces their (greedy) drafts.
// Other contexts: nothing.
int finish_best_paths(sdms_ctx* ctx, int32_t* draft_tok, int32_t* draft_len, float* draft_score, float* draft_edge_w,
                      cudaStream_t stream) {
  if (ctx->cfg.search_mode != 2 || ctx->dev.beam_stride == 0) return SDMS_OK;
  ++ctx->launches;
  return launch_best_path_fix(ctx->dev, draft_tok, draft_len, draft_score, draft_edge_w, stream) == cudaSuccess
             ? SDMS_OK : SDMS_ERR_CUDA;
}

template <class F>
int timed(sdms_ctx* ctx, int kernel, cudaStream_t stream, F launch) {
  EventPair ev{};
  if (ctx->profiling) {
    if (!ctx->pool.empty()) { ev = ctx->pool.back(); ctx->pool.pop_back(); }
    else {
      if (cudaEventCreate(&ev.a) != cudaSuccess) return SDMS_ERR_CUDA;
      if (cudaEventCreate(&ev.b) != cudaSuccess) { cudaEventDestroy(ev.a); return SDMS_ERR_CUDA; }
    }
    ev.kernel = kernel;
    cudaEventRecord(ev.a, stream);
  }
  const cudaError_t e = launch();
  ++ctx->launches;
  if (ctx->profiling) {
    cudaEventRecord(ev.b, stream);
    ctx->pending.push_back(ev);
    if (ctx->pending.size() >= kMaxPendingEvents) drain_pending(ctx, kMaxPendingEvents / 2);   // a long loop that never reads
  }
  return e == cudaSuccess ? SDMS_OK : SDMS_ERR_CUDA;
}

}  // namespace

extern "C" {

int sdms_workspace_bytes(const sdms_config* cfg, size_t* bytes) {
  if (!bytes) return SDMS_ERR_INVALID_ARG;
  Layout lay;
  const int rc = check_all(cfg, &lay);
  if (rc != SDMS_OK) return rc;
  *bytes = lay.total;
  return SDMS_OK;
}

int sdms_create(const sdms_config* cfg, void* d_workspace, size_t bytes, sdms_ctx** out) {
  if (!out) return SDMS_ERR_INVALID_ARG;
  *out = nullptr;
  Layout lay;
  const int rc = check_all(cfg, &lay);
  if (rc != SDMS_OK) return rc;
  if (!d_workspace || ((uintptr_t)d_workspace & (kAlign - 1))) return SDMS_ERR_INVALID_ARG;
  if (bytes < lay.total) return SDMS_ERR_WORKSPACE_TOO_SMALL;
  if (dag_kernel_setup() != cudaSuccess || scan_kernel_setup() != cudaSuccess) return SDMS_ERR_CUDA;
  if (cudaMemsetAsync(d_workspace, 0, lay.total, 0) != cudaSuccess) return SDMS_ERR_CUDA;
  if (cudaStreamSynchronize(0) != cudaSuccess) return SDMS_ERR_CUDA;
  sdms_ctx* ctx = new (std::nothrow) sdms_ctx();
  if (!ctx) return SDMS_ERR_BAD_STATE;
  ctx->cfg = *cfg;
  ctx->lay = lay;
  ctx->ws = static_cast<unsigned char*>(d_workspace);
  ctx->launches = 0;
  ctx->profiling = false;
  ctx->built = false;
  std::memset(ctx->prof_ms, 0, sizeof(ctx->prof_ms));
  std::memset(ctx->prof_n, 0, sizeof(ctx->prof_n));
  Dev& d = ctx->dev;
  d.G = cfg->num_groups; d.N = cfg->paths_per_group; d.L = cfg->capacity; d.V = cfg->vocab;
  d.k_max = cfg->k_max; d.idx_n = cfg->index_max_n ? cfg->index_max_n : cfg->k_max; d.D = cfg->max_draft_len; d.max_append = cfg->max_append;
  d.B = cfg->dag_nodes_per_layer; d.Ke = cfg->dag_nodes_per_layer ? cfg->dag_edges_per_node : 0;
  d.mode = cfg->search_mode; d.P = d.G * d.N;
  d.alpha = (double)cfg->alpha;
  d.table_cap = lay.table_cap; d.match_cap = lay.match_cap;
  {
    int l = 0;
    while ((1ll << l) < (long long)d.L) ++l;                          // l = ceil(log2 L)
    const unsigned long long two = 1ull << (31 + l);
    d.L_magic = (uint32_t)((two + (unsigned long long)d.L - 1) / (unsigned long long)d.L);
    d.L_shift = 31 + l;
  }
  d.fused = fits_fused(cfg, lay);
  d.eps = cfg->epsilon;
  d.pool = cfg->pool_mode;
  d.R = cfg->max_matches_per_path;
  ctx->step_fits = false;                        // decided below, once the kernels' attributes are set
  unsigned char* w = ctx->ws;
  d.tok = (int32_t*)(w + lay.tok); d.pq = (int32_t*)(w + lay.pq); d.len = (int32_t*)(w + lay.len); d.rec = (int32_t*)(w + lay.rec);
  d.status = (uint32_t*)(w + lay.status); d.index = (uint32_t*)(w + lay.index);
  d.q_fp = (uint32_t*)(w + lay.q_fp); d.q_mode = (int32_t*)(w + lay.q_mode);
  d.q_reserved = (int32_t*)(w + lay.q_reserved); d.q_off = (int32_t*)(w + lay.q_off);
  d.match_cursor = (unsigned long long*)(w + lay.match_cursor);
  d.q_cursor = (int32_t*)(w + lay.q_cursor); d.g_nscan = (int32_t*)(w + lay.g_nscan); d.g_trim = (int32_t*)(w + lay.g_trim);
  d.matches = (int32_t*)(w + lay.matches);
  ctx->x_draft_tok = (int32_t*)(w + lay.x_draft_tok); ctx->x_draft_len = (int32_t*)(w + lay.x_draft_len);
  d.x_node_tok = (int32_t*)(w + lay.x_node_tok); d.x_node_S = (int64_t*)(w + lay.x_node_S);
  d.x_node_cnt = (int32_t*)(w + lay.x_node_cnt); d.x_node_count = (int32_t*)(w + lay.x_node_count);
  d.x_edge_dst = (int32_t*)(w + lay.x_edge_dst); d.x_edge_S = (int64_t*)(w + lay.x_edge_S);
  d.x_edge_cnt = (int32_t*)(w + lay.x_edge_cnt); d.x_out_degree = (int32_t*)(w + lay.x_out_degree);
  d.w_ctl = (unsigned long long*)(w + lay.w_ctl); d.w_desc = (int4*)(w + lay.w_desc);
  d.w_pred = (WidePred*)(w + lay.w_pred); d.w_edge = (unsigned long long*)(w + lay.w_edge);
  d.w_tab = (WideSlot*)(w + lay.w_tab); d.w_key = (uint32_t*)(w + lay.w_key); d.w_item = (int32_t*)(w + lay.w_item);
  d.w_grid = lay.wide_on ? wide_kernel_grid() : 0;   // 0 (also without cooperative launch on this device): one thread block per query
  d.w_slots = lay.w_slots;
  d.b_ent = (BeamEnt*)(w + lay.b_ent); d.b_ctl = (unsigned long long*)(w + lay.b_ctl); d.bp_todo = (int32_t*)(w + lay.bp_todo); d.beam_stride = lay.w_slots ? (cfg->max_beams > 0 ? cfg->max_beams : (cfg->search_mode == 2 ? 1 : 0)) : 0;
  ctx->step_fits = step_kernel_fits(d);
  d.build_cluster = build_cluster_size(d);
  *out = ctx;
  return SDMS_OK;
}

int sdms_reset(sdms_ctx* ctx, void* stream) {
  if (!ctx) return SDMS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  // the path store need not be cleared: lengths say what is valid
  const Layout& l = ctx->lay;
  if (cudaMemsetAsync(ctx->ws + l.len, 0, l.matches - l.len, st) != cudaSuccess) return SDMS_ERR_CUDA;
  ctx->built = false;
  return SDMS_OK;
}

int sdms_destroy(sdms_ctx* ctx) {
  if (!ctx) return SDMS_ERR_INVALID_ARG;
  for (auto& e : ctx->pending) { cudaEventDestroy(e.a); cudaEventDestroy(e.b); }
  for (auto& e : ctx->pool) { cudaEventDestroy(e.a); cudaEventDestroy(e.b); }
  delete ctx;
  return SDMS_OK;
}

int sdms_append(sdms_ctx* ctx, const int32_t* d_tokens, const float* d_logprobs, const int32_t* d_counts,
                int32_t row_width, void* stream) {
  if (!ctx || !d_tokens || !d_logprobs || !d_counts || row_width < 1) return SDMS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  ctx->built = false;
  return timed(ctx, SDMS_KERNEL_APPEND, st,
               [&] { return launch_append(ctx->dev, d_tokens, d_logprobs, d_counts, row_width, st); });
}

int sdms_build_drafts(sdms_ctx* ctx, int32_t k, int32_t* d_draft_tok, int32_t* d_draft_len,
                      float* d_draft_score, float* d_draft_edge_w, void* stream) {
  if (!ctx || !d_draft_tok || !d_draft_len) return SDMS_ERR_INVALID_ARG;
  if (k < 1 || k > ctx->cfg.k_max) return SDMS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (ctx->dev.fused) {
    const int rc = timed(ctx, SDMS_KERNEL_BUILD_FUSED, st, [&] {
      return launch_build_fused(ctx->dev, k, k, d_draft_tok, d_draft_len, d_draft_score, d_draft_edge_w, nullptr, st); });
    if (rc != SDMS_OK) return rc;
    ctx->built = true;
    return finish_best_paths(ctx, d_draft_tok, d_draft_len, d_draft_score, d_draft_edge_w, st);
  }
  int rc;
  if (ctx->dev.eps > 0) {                            // matches with tolerance: sized by counting, four launches
    rc = timed(ctx, SDMS_KERNEL_SCAN, st, [&] { return launch_fuzzy_match(ctx->dev, k, 0, st); });
    ctx->launches += 3;
  } else {
    rc = timed(ctx, SDMS_KERNEL_PROBE, st, [&] { return launch_probe(ctx->dev, k, 0, st); });
    if (rc != SDMS_OK) return rc;
    rc = timed(ctx, SDMS_KERNEL_SCAN, st, [&] { return launch_scan(ctx->dev, k, st); });
  }
  if (rc != SDMS_OK) return rc;
  rc = timed(ctx, SDMS_KERNEL_DAG, st, [&] {
    return launch_dag(ctx->dev, false, d_draft_tok, d_draft_len, d_draft_score, d_draft_edge_w, st); });
  if (rc == SDMS_OK && ctx->dev.w_grid > 0)
    rc = timed(ctx, SDMS_KERNEL_DAG_WIDE, st, [&] {
      return launch_dag_wide(ctx->dev, d_draft_tok, d_draft_len, d_draft_score, d_draft_edge_w, st); });
  if (rc != SDMS_OK) return rc;
  ctx->built = true;
  return finish_best_paths(ctx, d_draft_tok, d_draft_len, d_draft_score, d_draft_edge_w, st);
}

int sdms_build_drafts_backoff(sdms_ctx* ctx, int32_t k_hi, int32_t* d_draft_tok, int32_t* d_draft_len,
                              float* d_draft_score, float* d_draft_edge_w, int32_t* d_used_k, void* stream) {
  if (!ctx || !d_draft_tok || !d_draft_len) return SDMS_ERR_INVALID_ARG;
  if (k_hi < 1 || k_hi > ctx->cfg.k_max) return SDMS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (!ctx->dev.fused) {
    // large prompts: one probe / scan / dag (/ wide) round per suffix length, longest first; a path that has found
    // matches keeps them and its draft, the others try again with a shorter suffix
    for (int k = k_hi; k >= 1; --k) {
      const int round = kRoundBackoff | (k < k_hi ? kRoundNotFirst : 0) | (k == 1 ? kRoundLast : 0);
      int rc;
      if (ctx->dev.eps > 0) {
        rc = timed(ctx, SDMS_KERNEL_SCAN, st, [&] { return launch_fuzzy_match(ctx->dev, k, k < k_hi, st); });
        ctx->launches += 3;
      } else {
        rc = timed(ctx, SDMS_KERNEL_PROBE, st, [&] { return launch_probe(ctx->dev, k, k < k_hi, st); });
        if (rc == SDMS_OK) rc = timed(ctx, SDMS_KERNEL_SCAN, st, [&] { return launch_scan(ctx->dev, k, st); });
      }
      if (rc == SDMS_OK)
        rc = timed(ctx, SDMS_KERNEL_DAG, st, [&] {
          return launch_dag(ctx->dev, false, d_draft_tok, d_draft_len, d_draft_score, d_draft_edge_w, st, round, k, d_used_k); });
      if (rc == SDMS_OK && ctx->dev.w_grid > 0)
        rc = timed(ctx, SDMS_KERNEL_DAG_WIDE, st, [&] {
          return launch_dag_wide(ctx->dev, d_draft_tok, d_draft_len, d_draft_score, d_draft_edge_w, st); });
      if (rc != SDMS_OK) return rc;
      rc = finish_best_paths(ctx, d_draft_tok, d_draft_len, d_draft_score, d_draft_edge_w, st);
      if (rc != SDMS_OK) return rc;
    }
    ctx->built = true;
    return SDMS_OK;
  }
  const int rc = timed(ctx, SDMS_KERNEL_BUILD_FUSED, st, [&] {
    return launch_build_fused(ctx->dev, k_hi, 1, d_draft_tok, d_draft_len, d_draft_score, d_draft_edge_w, d_used_k, st); });
  if (rc != SDMS_OK) return rc;
  ctx->built = true;
  return finish_best_paths(ctx, d_draft_tok, d_draft_len, d_draft_score, d_draft_edge_w, st);
}

int sdms_accept(sdms_ctx* ctx, const int32_t* d_draft_tok, const int32_t* d_draft_len, const int32_t* d_sampled,
                const float* d_sampled_logprobs, int32_t* d_accept_len, void* stream) {
  if (!ctx || !d_draft_tok || !d_draft_len || !d_sampled || !d_accept_len) return SDMS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (d_sampled_logprobs) ctx->built = false;          // the commit changes the histories
  return timed(ctx, SDMS_KERNEL_ACCEPT, st, [&] {
    return launch_accept(ctx->dev, d_draft_tok, d_draft_len, d_sampled, d_sampled_logprobs, d_accept_len, st); });
}

int sdms_trim(sdms_ctx* ctx, const int32_t* d_keep, void* stream) {
  if (!ctx || !d_keep) return SDMS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  ctx->built = false;
  if (cudaMemsetAsync(ctx->dev.g_trim, 0, (size_t)ctx->dev.G * 4, st) != cudaSuccess) return SDMS_ERR_CUDA;
  for (int phase = 0; phase < 3; ++phase) {
    const int rc = timed(ctx, SDMS_KERNEL_TRIM, st, [&] { return launch_trim(ctx->dev, phase, d_keep, st); });
    if (rc != SDMS_OK) return rc;
  }
  return SDMS_OK;
}

int sdms_step(sdms_ctx* ctx, int32_t k, const int32_t* d_sampled, const float* d_sampled_logprobs,
              int32_t* d_accept_len, int32_t* d_draft_tok, int32_t* d_draft_len, float* d_draft_score,
              float* d_draft_edge_w, void* stream) {
  if (!ctx || !d_sampled || !d_sampled_logprobs || !d_accept_len || !d_draft_tok || !d_draft_len)
    return SDMS_ERR_INVALID_ARG;
  if (k < 1 || k > ctx->cfg.k_max) return SDMS_ERR_INVALID_ARG;
  if (!ctx->step_fits) {
    const int rc = sdms_accept(ctx, d_draft_tok, d_draft_len, d_sampled, d_sampled_logprobs, d_accept_len, stream);
    if (rc != SDMS_OK) return rc;
    return sdms_build_drafts(ctx, k, d_draft_tok, d_draft_len, d_draft_score, d_draft_edge_w, stream);
  }
  cudaStream_t st = (cudaStream_t)stream;
  ctx->built = false;
  const int rc = timed(ctx, SDMS_KERNEL_STEP, st, [&] {
    return launch_step(ctx->dev, k, k, d_sampled, d_sampled_logprobs, d_accept_len, d_draft_tok, d_draft_len,
                       d_draft_score, d_draft_edge_w, nullptr, st); });
  if (rc != SDMS_OK) return rc;
  ctx->built = true;
  return finish_best_paths(ctx, d_draft_tok, d_draft_len, d_draft_score, d_draft_edge_w, st);
}

int sdms_step_backoff(sdms_ctx* ctx, int32_t k_hi, const int32_t* d_sampled, const float* d_sampled_logprobs,
                      int32_t* d_accept_len, int32_t* d_draft_tok, int32_t* d_draft_len, float* d_draft_score,
                      float* d_draft_edge_w, int32_t* d_used_k, void* stream) {
  if (!ctx || !d_sampled || !d_sampled_logprobs || !d_accept_len || !d_draft_tok || !d_draft_len)
    return SDMS_ERR_INVALID_ARG;
  if (k_hi < 1 || k_hi > ctx->cfg.k_max) return SDMS_ERR_INVALID_ARG;
  if (!ctx->step_fits) {
    const int rc = sdms_accept(ctx, d_draft_tok, d_draft_len, d_sampled, d_sampled_logprobs, d_accept_len, stream);
    if (rc != SDMS_OK) return rc;
    return sdms_build_drafts_backoff(ctx, k_hi, d_draft_tok, d_draft_len, d_draft_score, d_draft_edge_w, d_used_k,
                                     stream);
  }
  cudaStream_t st = (cudaStream_t)stream;
  ctx->built = false;
  const int rc = timed(ctx, SDMS_KERNEL_STEP, st, [&] {
    return launch_step(ctx->dev, k_hi, 1, d_sampled, d_sampled_logprobs, d_accept_len, d_draft_tok, d_draft_len,
                       d_draft_score, d_draft_edge_w, d_used_k, st); });
  if (rc != SDMS_OK) return rc;
  ctx->built = true;
  return finish_best_paths(ctx, d_draft_tok, d_draft_len, d_draft_score, d_draft_edge_w, st);
}

int sdms_step_is_single_launch(sdms_ctx* ctx, int32_t* yes) {
  if (!ctx || !yes) return SDMS_ERR_INVALID_ARG;
  *yes = ctx->step_fits ? 1 : 0;
  return SDMS_OK;
}

int sdms_build_cluster_size(sdms_ctx* ctx, int32_t* paths) {
  if (!ctx || !paths) return SDMS_ERR_INVALID_ARG;
  *paths = ctx->dev.build_cluster > 1 ? ctx->dev.build_cluster : 1;
  return SDMS_OK;
}

int sdms_host_pointer(const void* host_ptr, void** device_ptr) {
  if (!host_ptr || !device_ptr) return SDMS_ERR_INVALID_ARG;
  cudaPointerAttributes a{};
  if (cudaPointerGetAttributes(&a, host_ptr) != cudaSuccess) { cudaGetLastError(); return SDMS_ERR_INVALID_ARG; }
  if (a.type != cudaMemoryTypeHost || !a.devicePointer) return SDMS_ERR_INVALID_ARG;
  *device_ptr = a.devicePointer;
  return SDMS_OK;
}

int sdms_get_matches(sdms_ctx* ctx, int32_t* d_offsets, int32_t* d_gpos, size_t cap, void* stream) {
  if (!ctx || !d_offsets || (!d_gpos && cap)) return SDMS_ERR_INVALID_ARG;
  if (!ctx->built) return SDMS_ERR_BAD_STATE;
  const cudaError_t e = launch_compact_matches(ctx->dev, d_offsets, d_gpos, cap, (cudaStream_t)stream);
  ++ctx->launches;
  return e == cudaSuccess ? SDMS_OK : SDMS_ERR_CUDA;
}

int sdms_get_dag(sdms_ctx* ctx, int32_t* d_node_tok, int64_t* d_node_S, int32_t* d_node_cnt,
                 int32_t* d_node_count, int32_t* d_edge_dst, int64_t* d_edge_S, int32_t* d_edge_cnt,
                 int32_t* d_out_degree, void* stream) {
  if (!ctx) return SDMS_ERR_INVALID_ARG;
  if (!ctx->built || ctx->dev.B == 0) return SDMS_ERR_BAD_STATE;
  cudaStream_t st = (cudaStream_t)stream;
  const Dev& d = ctx->dev;
  const size_t nb = (size_t)d.P * d.D * d.B, ne = nb * d.Ke;
  // aggregate again over the matches of the last build, this time keeping the ranked nodes and edges
  const int rc = timed(ctx, SDMS_KERNEL_DAG, st, [&] {
    return launch_dag(d, true, ctx->x_draft_tok, ctx->x_draft_len, nullptr, nullptr, st); });
  if (rc != SDMS_OK) return rc;
  bool ok = true;
  auto copy = [&](void* dst, const void* src, size_t bytes) {
    if (dst && bytes) ok = ok && cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  };
  copy(d_node_tok, d.x_node_tok, nb * 4); copy(d_node_S, d.x_node_S, nb * 8); copy(d_node_cnt, d.x_node_cnt, nb * 4);
  copy(d_node_count, d.x_node_count, (size_t)d.P * d.D * 4);
  copy(d_edge_dst, d.x_edge_dst, ne * 4); copy(d_edge_S, d.x_edge_S, ne * 8); copy(d_edge_cnt, d.x_edge_cnt, ne * 4);
  copy(d_out_degree, d.x_out_degree, nb * 4);
  return ok ? SDMS_OK : SDMS_ERR_CUDA;
}

int sdms_get_beams(sdms_ctx* ctx, int32_t num_beams, int32_t* d_beam_tok, int32_t* d_beam_len, float* d_beam_value,
                   void* stream) {
  if (!ctx || !d_beam_tok || !d_beam_len || !d_beam_value) return SDMS_ERR_INVALID_ARG;
  if (num_beams < 1 || num_beams > SDMS_MAX_BEAMS) return SDMS_ERR_INVALID_ARG;
  if (!ctx->built || num_beams > ctx->cfg.max_beams || ctx->dev.w_slots == 0) return SDMS_ERR_BAD_STATE;
  const cudaError_t e = launch_beams(ctx->dev, num_beams, d_beam_tok, d_beam_len, d_beam_value, (cudaStream_t)stream);
  ++ctx->launches;
  return e == cudaSuccess ? SDMS_OK : SDMS_ERR_CUDA;
}

int sdms_debug_read_history(sdms_ctx* ctx, int32_t* d_tok, int32_t* d_pq, int32_t* d_len, void* stream) {
  if (!ctx) return SDMS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const Dev& d = ctx->dev;
  const size_t n = (size_t)d.P * d.L * 4;
  bool ok = true;
  if (d_tok) ok = ok && cudaMemcpyAsync(d_tok, d.tok, n, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  if (d_pq) ok = ok && cudaMemcpyAsync(d_pq, d.pq, n, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  if (d_len) ok = ok && cudaMemcpyAsync(d_len, d.len, (size_t)d.P * 4, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  return ok ? SDMS_OK : SDMS_ERR_CUDA;
}

int sdms_debug_read_query_modes(sdms_ctx* ctx, int32_t* d_modes, void* stream) {
  if (!ctx || !d_modes) return SDMS_ERR_INVALID_ARG;
  if (!ctx->built) return SDMS_ERR_BAD_STATE;
  return cudaMemcpyAsync(d_modes, ctx->dev.q_mode, (size_t)ctx->dev.P * 4, cudaMemcpyDeviceToDevice,
                         (cudaStream_t)stream) == cudaSuccess ? SDMS_OK : SDMS_ERR_CUDA;
}

int sdms_debug_wait_timeout(sdms_ctx* ctx, void* stream) {
  if (!ctx) return SDMS_ERR_INVALID_ARG;
  ++ctx->launches;
  return launch_wait_timeout(ctx->dev, 1000000LL, (cudaStream_t)stream) == cudaSuccess ? SDMS_OK : SDMS_ERR_CUDA;
}

int sdms_get_status(sdms_ctx* ctx, uint32_t* host_flags, void* stream) {
  if (!ctx || !host_flags) return SDMS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(host_flags, ctx->dev.status, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return SDMS_ERR_CUDA;
  if (cudaMemsetAsync(ctx->dev.status, 0, 4, st) != cudaSuccess) return SDMS_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return SDMS_ERR_CUDA;
  return SDMS_OK;
}

int sdms_launch_count(sdms_ctx* ctx, uint64_t* launches) {
  if (!ctx || !launches) return SDMS_ERR_INVALID_ARG;
  *launches = ctx->launches;
  return SDMS_OK;
}

int sdms_profile_enable(sdms_ctx* ctx, int32_t on) {
  if (!ctx) return SDMS_ERR_INVALID_ARG;
  ctx->profiling = on != 0;
  return SDMS_OK;
}

int sdms_profile_read(sdms_ctx* ctx, float* ms, uint64_t* launches) {
  if (!ctx || !ms || !launches) return SDMS_ERR_INVALID_ARG;
  const int rc = drain_pending(ctx, ctx->pending.size());
  if (rc != SDMS_OK) return rc;
  for (int k = 0; k < SDMS_NUM_KERNELS; ++k) {
    ms[k] = ctx->prof_ms[k]; launches[k] = ctx->prof_n[k];
    ctx->prof_ms[k] = 0.f; ctx->prof_n[k] = 0;
  }
  return SDMS_OK;
}

const char* sdms_strerror(int code) {
  switch (code) {
    case SDMS_OK: return "ok";
    case SDMS_ERR_INVALID_ARG: return "invalid argument";
    case SDMS_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case SDMS_ERR_CUDA: return "CUDA call failed";
    case SDMS_ERR_BAD_STATE: return "call not valid in this state";
    case SDMS_ERR_TOO_LARGE: return "size beyond the fixed maximum of this entry point";
    default: return "unknown error";
  }
}

const char* sdms_kernel_name(int kernel) {
  static const char* names[SDMS_NUM_KERNELS] = {"append", "probe", "scan", "dag", "accept", "build_fused", "step", "trim",
                                                "dag_wide"};
  return kernel >= 0 && kernel < SDMS_NUM_KERNELS ? names[kernel] : "?";
}

}  // extern "C"
