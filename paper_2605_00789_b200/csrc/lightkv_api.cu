// liblightkv C ABI: plan (host only), argument validation, kernel sequencing.
#include <math.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <vector>

#include "launch.h"

namespace lkv {

struct StagePlan {
  int layer, w;
  double keep;
  int cap_in, cap_out, cap_a, cap_b, n_windows;
  bool exact;      // cap_in is the exact count (schedule so far is data independent)
  bool exact_out;  // cap_out too
  bool use_tc;
  int fd_tiles;    // estimate of the tiles per sample of the tensor-core FD kernel (sizes its launch)
  Geometry geo;
  size_t ws_bytes;
  size_t off[16];     // byte offsets of the Workspace arrays
};

}  // namespace lkv

struct lightkv_plan {
  lightkv_config_t cfg;
  std::vector<lightkv_tile_t> tiles;
  std::vector<lkv::StagePlan> stages;
  int n_vis0;
};

namespace lkv {

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Tiles per sample the window-build kernel reports when the largest window has max_a A entries (same
// rule as the kernel).  Only the launch shape of the persistent FD kernel depends on it, so an estimate
// is enough: the kernel itself walks whatever tiles the device-side tiling holds.
static int fd_tile_count(int n_windows, int max_a, int batch) {
  if (max_a <= 0) return 0;
  if (max_a <= kFdTile) {
    const int want = (n_windows * batch + kFdTargetTiles - 1) / kFdTargetTiles;
    const int wpt = std::max(1, std::min(std::min(kFdTile / max_a, n_windows), want));
    return (n_windows + wpt - 1) / wpt;
  }
  const int blocks = (max_a + kFdTile - 1) / kFdTile;
  return n_windows * blocks * blocks;
}

static void layout_workspace(const lightkv_plan_t& p, StagePlan& s) {
  const size_t B = p.cfg.batch, nW1 = s.n_windows + 1;
  const bool attn = p.cfg.xi_mode == LIGHTKV_XI_ATTN_FULL || p.cfg.xi_mode == LIGHTKV_XI_ATTN_LSE;
  const size_t xi_items = attn ? size_t((s.cap_in + 127) / 128) * p.cfg.n_q_heads * B : 0;
  const size_t sizes[16] = {
      B * nW1 * 4, B * nW1 * 4, B * s.cap_in * 4, B * s.cap_in * 4, B * s.cap_a * 4, B * s.cap_a * 4,
      B * s.cap_b * 4, B * s.cap_a * 8, B * sizeof(FdTiling),
      attn ? B * p.cfg.n_q_heads * s.cap_in * 4 : 0, B * s.cap_in * 4, B * s.cap_in * 4, B * s.cap_in * 4,
      B * s.cap_a * 4, attn ? size_t(16) : size_t(0), xi_items * 4};
  size_t off = 0;
  for (int i = 0; i < 16; ++i) { s.off[i] = off; off += align_up(sizes[i], 256); }
  s.ws_bytes = std::max<size_t>(off, 256);
}

static Workspace bind_workspace(const StagePlan& s, void* base) {
  char* p = static_cast<char*>(base);
  Workspace w;
  w.win_off = reinterpret_cast<int*>(p + s.off[0]);
  w.a_off = reinterpret_cast<int*>(p + s.off[1]);
  w.tok_win = reinterpret_cast<int*>(p + s.off[2]);
  w.tok_l = reinterpret_cast<int*>(p + s.off[3]);
  w.a_tok = reinterpret_cast<int*>(p + s.off[4]);
  w.a_win = reinterpret_cast<int*>(p + s.off[5]);
  w.b_tok = reinterpret_cast<int*>(p + s.off[6]);
  w.a_key = reinterpret_cast<unsigned long long*>(p + s.off[7]);
  w.fd_tiling = reinterpret_cast<FdTiling*>(p + s.off[8]);
  w.xi_h = reinterpret_cast<float*>(p + s.off[9]);
  w.xi = reinterpret_cast<float*>(p + s.off[10]);
  w.partner = reinterpret_cast<int*>(p + s.off[11]);
  w.slot = reinterpret_cast<int*>(p + s.off[12]);
  w.a_partner = reinterpret_cast<int*>(p + s.off[13]);
  w.xi_sched = reinterpret_cast<unsigned int*>(p + s.off[14]);
  w.xi_redo = reinterpret_cast<int*>(p + s.off[15]);
  w.cap_in = s.cap_in; w.cap_out = s.cap_out; w.cap_a = s.cap_a; w.cap_b = s.cap_b;
  w.n_windows = s.n_windows;
  return w;
}

}  // namespace lkv

using namespace lkv;

extern "C" {

int lightkv_version(void) { return LIGHTKV_VERSION; }

const char* lightkv_status_string(int status) {
  switch (status) {
    case LIGHTKV_OK: return "ok";
    case LIGHTKV_ERR_INVALID_ARG: return "invalid argument";
    case LIGHTKV_ERR_UNSUPPORTED: return "unsupported configuration";
    case LIGHTKV_ERR_WORKSPACE: return "workspace too small or misaligned";
    case LIGHTKV_ERR_CAPACITY: return "capacity exceeded";
    case LIGHTKV_ERR_CUDA: return "CUDA error";
    case LIGHTKV_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

int lightkv_plan(const lightkv_config_t* c, lightkv_plan_t** out) {
  if (!c || !out) return LIGHTKV_ERR_INVALID_ARG;
  *out = nullptr;
  if (c->struct_size != sizeof(lightkv_config_t)) return LIGHTKV_ERR_INVALID_ARG;
  if (c->batch <= 0 || c->hidden <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->head_dim <= 0 ||
      c->n_layers <= 0 || c->n_tiles <= 0 || c->n_stages <= 0 || c->max_text < 0)
    return LIGHTKV_ERR_INVALID_ARG;
  if (!c->tiles || !c->layers || !c->windows || !c->keep) return LIGHTKV_ERR_INVALID_ARG;
  if (c->hidden % 8 || c->head_dim % 8 || c->n_q_heads % c->n_kv_heads) return LIGHTKV_ERR_INVALID_ARG;
  if (c->dtype != LIGHTKV_BF16 && c->dtype != LIGHTKV_FP32) return LIGHTKV_ERR_INVALID_ARG;
  if (c->xi_mode < LIGHTKV_XI_GIVEN || c->xi_mode > LIGHTKV_XI_UNIFORM) return LIGHTKV_ERR_INVALID_ARG;
  if (c->engine != LIGHTKV_ENGINE_AUTO && c->engine != LIGHTKV_ENGINE_SIMT) return LIGHTKV_ERR_INVALID_ARG;
  if (c->ragged_input != 0 && c->ragged_input != 1) return LIGHTKV_ERR_INVALID_ARG;
  if (c->divergence < LIGHTKV_FD_COSINE || c->divergence > LIGHTKV_FD_L2) return LIGHTKV_ERR_INVALID_ARG;
  if (c->direction != LIGHTKV_DIR_A2B && c->direction != LIGHTKV_DIR_B2A) return LIGHTKV_ERR_INVALID_ARG;
  if (c->n_tiles > kMaxTiles) return LIGHTKV_ERR_UNSUPPORTED;
  if (c->head_dim > 256) return LIGHTKV_ERR_UNSUPPORTED;

  lightkv_plan_t* p = new (std::nothrow) lightkv_plan_t;
  if (!p) return LIGHTKV_ERR_INVALID_ARG;
  p->cfg = *c;
  p->tiles.assign(c->tiles, c->tiles + c->n_tiles);
  p->cfg.tiles = nullptr; p->cfg.layers = nullptr; p->cfg.windows = nullptr; p->cfg.keep = nullptr;
  long long n_vis = 0;
  for (const auto& t : p->tiles) {
    if (t.rows <= 0 || t.cols <= 0) { delete p; return LIGHTKV_ERR_INVALID_ARG; }
    n_vis += (long long)t.rows * t.cols;
  }
  if (n_vis > (1 << 24)) { delete p; return LIGHTKV_ERR_UNSUPPORTED; }
  p->n_vis0 = (int)n_vis;

  // Host simulation of the schedule.  While every window either loses all of its A nodes or none,
  // the surviving positions do not depend on the data and the counts are exact.
  std::vector<int> alive(p->n_vis0);
  for (int i = 0; i < p->n_vis0; ++i) alive[i] = i;
  bool exact = c->ragged_input == 0;   // a subset of the grid makes every later count depend on the data
  int cap = p->n_vis0;
  for (int s = 0; s < c->n_stages; ++s) {
    StagePlan sp;
    memset(&sp, 0, sizeof(sp));
    sp.layer = c->layers[s]; sp.w = c->windows[s]; sp.keep = c->keep[s];
    if (sp.w <= 0 || !(sp.keep >= 0.5 && sp.keep <= 1.0) || sp.layer < 1 || sp.layer > c->n_layers ||
        (s > 0 && sp.layer <= c->layers[s - 1])) { delete p; return LIGHTKV_ERR_INVALID_ARG; }
    Geometry& g = sp.geo;
    g.n_tiles = c->n_tiles; g.w = sp.w; g.n_windows = c->n_tiles * sp.w * sp.w;
    g.src_par = c->direction == LIGHTKV_DIR_B2A ? 1 : 0;
    g.tile_off[0] = 0;
    for (int t = 0; t < c->n_tiles; ++t) {
      if (sp.w > p->tiles[t].rows || sp.w > p->tiles[t].cols) { delete p; return LIGHTKV_ERR_INVALID_ARG; }
      g.rows[t] = p->tiles[t].rows; g.cols[t] = p->tiles[t].cols;
      g.tile_off[t + 1] = g.tile_off[t] + g.rows[t] * g.cols[t];
    }
    if (g.n_windows > kMaxWindows) { delete p; return LIGHTKV_ERR_UNSUPPORTED; }
    // the window-build kernel counts the tokens of a window in 16 bits
    for (int t = 0; t < c->n_tiles; ++t)
      if ((long long)((g.rows[t] + sp.w - 1) / sp.w) * ((g.cols[t] + sp.w - 1) / sp.w) > kMaxWindowTokens) {
        delete p;
        return LIGHTKV_ERR_UNSUPPORTED;
      }
    sp.n_windows = g.n_windows;
    sp.cap_in = cap;
    sp.exact = exact;
    if (exact) {
      std::vector<std::vector<int>> members(g.n_windows);
      for (int pos : alive) members[window_of(g, pos)].push_back(pos);   // alive is ascending
      std::vector<int> next;
      int cap_a = 0, cap_b = 0, max_a = 0;
      bool still = true;
      for (const auto& m : members) {
        // sources: the tokens of local rank parity src_par; the others are the destinations and always survive
        const int n = (int)m.size(), na = (n + 1 - g.src_par) / 2, r = removal_count(n, sp.keep, g.src_par);
        cap_a += na; cap_b += n - na;
        max_a = std::max(max_a, std::max(na, n - na));
        if (r == na && n >= 2) { for (int l = 1 - g.src_par; l < n; l += 2) next.push_back(m[l]); }
        else if (r == 0) { next.insert(next.end(), m.begin(), m.end()); }
        else still = false;
      }
      sp.cap_a = cap_a; sp.cap_b = cap_b;
      sp.fd_tiles = fd_tile_count(g.n_windows, max_a, c->batch);
      if (still) {
        std::sort(next.begin(), next.end());
        alive.swap(next);
        sp.cap_out = (int)alive.size();
      } else {
        exact = false;
      }
    }
    if (!sp.exact) {      // sum over windows of ceil(n_w / 2) resp. floor(n_w / 2), whichever set is the source
      sp.cap_a = g.src_par ? sp.cap_in / 2 : (sp.cap_in + sp.n_windows) / 2;
      sp.cap_b = g.src_par ? (sp.cap_in + sp.n_windows) / 2 : sp.cap_in / 2;
    }
    if (!sp.exact) {  // counts depend on the data: a window holds at most the tokens of its grid cell
                      // (balanced cells: ceil(rows/w) x ceil(cols/w))
      int cell = 0;
      for (int t = 0; t < c->n_tiles; ++t)
        cell = std::max(cell, ((g.rows[t] + sp.w - 1) / sp.w) * ((g.cols[t] + sp.w - 1) / sp.w));
      sp.fd_tiles = fd_tile_count(g.n_windows, (std::min(cell, sp.cap_in) + 1) / 2, c->batch);
    }
    if (!exact) {   // data-dependent from here on: every window keeps at most ceil(keep n_w) tokens
      long long bound = (long long)ceil(sp.keep * sp.cap_in) + sp.n_windows;
      sp.cap_out = (int)std::min<long long>(bound, sp.cap_in);
    }
    sp.exact_out = exact;
    sp.cap_a = std::max(sp.cap_a, 1); sp.cap_b = std::max(sp.cap_b, 1);
    sp.use_tc = c->engine == LIGHTKV_ENGINE_AUTO && c->dtype == LIGHTKV_BF16;
    layout_workspace(*p, sp);
    cap = sp.cap_out;
    p->stages.push_back(sp);
  }
  // keep/layers/windows live in the stage plans
  *out = p;
  return LIGHTKV_OK;
}

int lightkv_plan_stage_info(const lightkv_plan_t* p, int32_t stage, lightkv_stage_info_t* info) {
  if (!p || !info || stage < 0 || stage >= (int)p->stages.size()) return LIGHTKV_ERR_INVALID_ARG;
  const StagePlan& s = p->stages[stage];
  info->layer = s.layer; info->window = s.w; info->keep = s.keep;
  info->cap_in = s.cap_in; info->cap_out = s.cap_out; info->n_windows = s.n_windows;
  info->counts_exact = (s.exact && s.exact_out) ? 1 : 0;
  info->uses_tensor_cores = (s.use_tc && (tc_fd_supported(p->cfg.hidden) ||
                                          ((p->cfg.xi_mode == LIGHTKV_XI_ATTN_FULL ||
                                            p->cfg.xi_mode == LIGHTKV_XI_ATTN_LSE) &&
                                           tc_xi_supported(p->cfg.head_dim)))) ? 1 : 0;
  info->workspace_bytes = s.ws_bytes;
  info->cap_a = s.cap_a; info->cap_b = s.cap_b; info->fd_tiles = s.fd_tiles; info->reserved = 0;
  return LIGHTKV_OK;
}

void lightkv_plan_destroy(lightkv_plan_t* p) { delete p; }

double lightkv_plan_retention(const lightkv_plan_t* p) {
  if (!p) return -1.0;
  // Eq. "complexity": lambda_1 + sum_i (lambda_i - lambda_{i-1}) prod_{j<i} keep_j + (L - lambda_s) prod keep_j
  double total = p->stages[0].layer, prod = 1.0;
  for (size_t i = 1; i < p->stages.size(); ++i) {
    prod *= p->stages[i - 1].keep;
    total += (p->stages[i].layer - p->stages[i - 1].layer) * prod;
  }
  prod *= p->stages.back().keep;
  total += (p->cfg.n_layers - p->stages.back().layer) * prod;
  return total / p->cfg.n_layers;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

int lightkv_compress_layer(const lightkv_plan_t* p, const lightkv_layer_args_t* a) {
  if (!p || !a || a->struct_size != sizeof(lightkv_layer_args_t)) return LIGHTKV_ERR_INVALID_ARG;
  if (a->stage < 0 || a->stage >= (int)p->stages.size()) return LIGHTKV_ERR_INVALID_ARG;
  const StagePlan& s = p->stages[a->stage];
  const lightkv_config_t& c = p->cfg;
  const size_t esz = c.dtype == LIGHTKV_BF16 ? 2 : 4;
  if (a->vis_begin < 0 || a->n_text_after < 0 || a->vis_begin + a->n_text_after > c.max_text)
    return LIGHTKV_ERR_INVALID_ARG;
  TextSet text;
  memset(&text, 0, sizeof(text));
  if (a->n_text_ranges < 0 || a->n_text_ranges > LIGHTKV_MAX_TEXT_RANGES) return LIGHTKV_ERR_INVALID_ARG;
  if (a->n_text_ranges == 0) {
    if (a->text_begin < 0 || a->text_end < a->text_begin || a->text_end > a->vis_begin) return LIGHTKV_ERR_INVALID_ARG;
    text.n = 1; text.lo[0] = a->text_begin; text.hi[0] = a->text_end;
  } else {
    if (!a->text_ranges) return LIGHTKV_ERR_INVALID_ARG;
    int prev_end = 0;
    for (int i = 0; i < a->n_text_ranges; ++i) {
      const int lo = a->text_ranges[2 * i], hi = a->text_ranges[2 * i + 1];
      if (lo < prev_end || hi < lo || hi > a->vis_begin) return LIGHTKV_ERR_INVALID_ARG;   // ascending, disjoint
      text.lo[i] = lo; text.hi[i] = hi;
      prev_end = hi;
    }
    text.n = a->n_text_ranges;
  }
  text.begin = text.lo[0]; text.end = text.hi[text.n - 1];
  if (a->bidirectional != 0 && a->bidirectional != 1) return LIGHTKV_ERR_INVALID_ARG;
  if (!a->hidden || !a->hidden_out || !a->n_vis_out || !a->pos_out || !a->dst || !a->weight || !a->grp_off ||
      !a->grp_src || !a->workspace)
    return LIGHTKV_ERR_INVALID_ARG;
  if (a->stage > 0 && !a->pos) return LIGHTKV_ERR_INVALID_ARG;       // identity positions only at stage 0
  if (a->hidden == a->hidden_out) return LIGHTKV_ERR_INVALID_ARG;
  if (!aligned16(a->hidden) || !aligned16(a->hidden_out) || (a->hidden_row_stride * esz) % 16 ||
      (a->hidden_out_row_stride * esz) % 16 || (a->hidden_batch_stride * esz) % 16 ||
      (a->hidden_out_batch_stride * esz) % 16 || a->hidden_row_stride < c.hidden ||
      a->hidden_out_row_stride < c.hidden)
    return LIGHTKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(a->workspace) & 255) != 0 || a->workspace_bytes < s.ws_bytes)
    return LIGHTKV_ERR_WORKSPACE;
  const bool attn = c.xi_mode == LIGHTKV_XI_ATTN_FULL || c.xi_mode == LIGHTKV_XI_ATTN_LSE;
  if (attn) {
    if (!a->q || !a->k || !aligned16(a->q) || !aligned16(a->k)) return LIGHTKV_ERR_INVALID_ARG;
    const int64_t st[6] = {a->q_batch_stride, a->q_head_stride, a->q_row_stride,
                           a->k_batch_stride, a->k_head_stride, a->k_row_stride};
    for (int64_t v : st) if ((v * (int64_t)esz) % 16) return LIGHTKV_ERR_INVALID_ARG;
    if (a->q_row_stride < c.head_dim || a->k_row_stride < c.head_dim) return LIGHTKV_ERR_INVALID_ARG;
    if (c.xi_mode == LIGHTKV_XI_ATTN_LSE && !a->lse) return LIGHTKV_ERR_INVALID_ARG;
  }
  if (c.xi_mode == LIGHTKV_XI_GIVEN && !a->xi) return LIGHTKV_ERR_INVALID_ARG;
  if (a->lse_out && c.xi_mode != LIGHTKV_XI_ATTN_FULL) return LIGHTKV_ERR_INVALID_ARG;
  if (a->aux_stream && (!a->fork_event || !a->join_event)) return LIGHTKV_ERR_INVALID_ARG;

  LayerLaunch L;
  L.batch = c.batch; L.hidden = c.hidden; L.n_q_heads = c.n_q_heads; L.n_kv_heads = c.n_kv_heads;
  L.head_dim = c.head_dim; L.dtype = c.dtype; L.xi_mode = c.xi_mode; L.divergence = c.divergence;
  L.keep = s.keep; L.geo = s.geo;
  L.fd_tiles = s.fd_tiles;
  L.ws = bind_workspace(s, a->workspace); L.text = text; L.a = a; L.stream = static_cast<cudaStream_t>(a->stream);

  cudaEvent_t* ev = reinterpret_cast<cudaEvent_t*>(a->trace_events);
  auto mark = [&](int i) { return ev ? cudaEventRecord(ev[i], L.stream) : cudaSuccess; };
  const bool tc_xi = s.use_tc && attn && tc_xi_supported(c.head_dim);
  const bool tc_fd = s.use_tc && tc_fd_supported(c.hidden);
  cudaStream_t aux = (a->aux_stream && attn && !ev) ? static_cast<cudaStream_t>(a->aux_stream) : nullptr;
  if (aux) {
    // fork: window build + FD (HBM bound) on the second stream, xi (bound by the exponentials) on the first.
    // The events are the caller's; once the fork is recorded the join is enqueued whatever happens between.
    cudaEvent_t fork = static_cast<cudaEvent_t>(a->fork_event), join = static_cast<cudaEvent_t>(a->join_event);
    LayerLaunch La = L;
    La.stream = aux;
    if (cudaEventRecord(fork, L.stream) != cudaSuccess) return LIGHTKV_ERR_CUDA;
    bool ok = cudaStreamWaitEvent(aux, fork, 0) == cudaSuccess;
    ok = ok && launch_window_build(La) == cudaSuccess;
    ok = ok && (tc_fd ? launch_fd_tc(La) : launch_fd_simt(La)) == cudaSuccess;
    const bool joined = cudaEventRecord(join, aux) == cudaSuccess;
    ok = ok && (tc_xi ? launch_xi_tc(L) : launch_xi_simt(L)) == cudaSuccess;
    const bool waited = joined && cudaStreamWaitEvent(L.stream, join, 0) == cudaSuccess;
    if (!ok || !waited) return LIGHTKV_ERR_CUDA;
  } else {
    if (mark(0) != cudaSuccess) return LIGHTKV_ERR_CUDA;
    if (launch_window_build(L) != cudaSuccess || mark(1) != cudaSuccess) return LIGHTKV_ERR_CUDA;
    if (attn && (tc_xi ? launch_xi_tc(L) : launch_xi_simt(L)) != cudaSuccess) return LIGHTKV_ERR_CUDA;
    if (mark(2) != cudaSuccess) return LIGHTKV_ERR_CUDA;
    if ((tc_fd ? launch_fd_tc(L) : launch_fd_simt(L)) != cudaSuccess || mark(3) != cudaSuccess)
      return LIGHTKV_ERR_CUDA;
  }
  if (launch_select_map(L) != cudaSuccess || mark(4) != cudaSuccess) return LIGHTKV_ERR_CUDA;
  if (a->map_event && cudaEventRecord(static_cast<cudaEvent_t>(a->map_event), L.stream) != cudaSuccess)
    return LIGHTKV_ERR_CUDA;
  if (launch_merge_rows(L) != cudaSuccess || mark(5) != cudaSuccess) return LIGHTKV_ERR_CUDA;
  return LIGHTKV_OK;
}

int lightkv_compact_kv(const lightkv_plan_t* p, const lightkv_kv_args_t* a) {
  if (!p || !a || a->struct_size != sizeof(lightkv_kv_args_t)) return LIGHTKV_ERR_INVALID_ARG;
  if (a->stage < 0 || a->stage >= (int)p->stages.size()) return LIGHTKV_ERR_INVALID_ARG;
  const StagePlan& s = p->stages[a->stage];
  const lightkv_config_t& c = p->cfg;
  const int64_t esz = c.dtype == LIGHTKV_BF16 ? 2 : 4;
  if (a->mode != LIGHTKV_KV_MERGE && a->mode != LIGHTKV_KV_GATHER) return LIGHTKV_ERR_INVALID_ARG;
  if (a->vis_begin < 0 || a->n_text_after < 0 || a->vis_begin + a->n_text_after > c.max_text)
    return LIGHTKV_ERR_INVALID_ARG;
  if (!a->n_vis_out || !a->grp_off || !a->grp_src || !a->weight || !a->k_src || !a->v_src || !a->k_dst ||
      !a->v_dst)
    return LIGHTKV_ERR_INVALID_ARG;
  // in place: K and V both, with one addressing (strides, page size, block tables) on the two sides
  const bool in_place = a->k_src == a->k_dst;
  if (in_place != (a->v_src == a->v_dst)) return LIGHTKV_ERR_INVALID_ARG;
  if (in_place && (a->src_batch_stride != a->dst_batch_stride || a->src_head_stride != a->dst_head_stride ||
                   a->src_row_stride != a->dst_row_stride || a->src_page_stride != a->dst_page_stride ||
                   (a->page_size > 0 && a->src_block_table != a->dst_block_table) ||
                   a->src_seq_start != a->dst_seq_start))
    return LIGHTKV_ERR_INVALID_ARG;
  const void* ptrs[4] = {a->k_src, a->v_src, a->k_dst, a->v_dst};
  for (const void* q : ptrs) if (!aligned16(q)) return LIGHTKV_ERR_INVALID_ARG;
  const int64_t st[8] = {a->src_batch_stride, a->src_head_stride, a->src_row_stride, a->src_page_stride,
                         a->dst_batch_stride, a->dst_head_stride, a->dst_row_stride, a->dst_page_stride};
  for (int64_t v : st) if ((v * esz) % 16) return LIGHTKV_ERR_INVALID_ARG;
  if (a->src_row_stride < c.head_dim || a->dst_row_stride < c.head_dim) return LIGHTKV_ERR_INVALID_ARG;
  if (a->page_size < 0) return LIGHTKV_ERR_INVALID_ARG;
  if (a->page_size > 0 && (!a->src_block_table || !a->dst_block_table || a->max_blocks <= 0 ||
      (long long)a->max_blocks * a->page_size < (long long)a->vis_begin + s.cap_in + a->n_text_after))
    return LIGHTKV_ERR_INVALID_ARG;
  KvLaunch K;
  K.batch = c.batch; K.n_kv_heads = c.n_kv_heads; K.head_dim = c.head_dim; K.dtype = c.dtype;
  K.cap_in = s.cap_in; K.cap_out = s.cap_out; K.a = a; K.stream = static_cast<cudaStream_t>(a->stream);
  if (launch_kv_compact(K) != cudaSuccess) return LIGHTKV_ERR_CUDA;
  return LIGHTKV_OK;
}

}  // extern "C"
