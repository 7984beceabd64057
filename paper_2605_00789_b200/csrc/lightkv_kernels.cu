// liblightkv kernels, part 1: window build, fp32-FMA contractions (FD, xi), selection + merge map,
// weighted merge of hidden states, K/V merge-compaction.  sm_100a.
#include <algorithm>

#include "launch.h"
#include "tc_common.cuh"

namespace lkv {

__device__ inline void set_status(uint32_t* status, uint32_t bit) {
  if (status) atomicOr(status, bit);
}

// =====================================================================================================
// Window build ("Window partitioning", Step 1).  One CTA per sample.
// Every token gets its window id from its original grid position; tokens of a window are ranked in
// storage order (positions ascend with storage, so this is position order).  Rank l even -> set A
// (the paper's 1st, 3rd, ... token), odd -> set B.  The SOURCE nodes (the ones that may be merged away: set A,
// or set B in the reverse direction, g.src_par = 1) go to the a_* lists, the destinations to b_tok, window by
// window.
// Stable ranking without sorting: each warp owns a contiguous segment of the tokens and a private row
// of per-window counters; an exclusive prefix over the 32 rows gives every warp its starting rank.
// =====================================================================================================
__global__ void __launch_bounds__(1024)
window_build_kernel(Geometry g, const int* __restrict__ pos_all, const int* __restrict__ n_vis,
                    Workspace ws, uint32_t* status) {
  grid_dependency_sync();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int nW = g.n_windows;
  uint16_t* cnt = reinterpret_cast<uint16_t*>(smem_raw);                        // [32][nW]
  int* wsum = reinterpret_cast<int*>(smem_raw + ((size_t(32) * nW * 2 + 15) & ~size_t(15)));  // [nW+1]
  int* asum = wsum + nW + 1;                                                    // [nW+1]

  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wp = tid >> 5;
  int n = n_vis ? n_vis[b] : ws.cap_in;
  if (n > ws.cap_in) { n = ws.cap_in; if (tid == 0) set_status(status, LIGHTKV_STATUS_COUNT); }
  if (n < 0) n = 0;
  const int* pos = pos_all ? pos_all + size_t(b) * ws.cap_in : nullptr;
  int* tok_win = ws.tok_win + size_t(b) * ws.cap_in;
  int* tok_l = ws.tok_l + size_t(b) * ws.cap_in;
  int* a_tok = ws.a_tok + size_t(b) * ws.cap_a;
  int* a_win = ws.a_win + size_t(b) * ws.cap_a;
  int* b_tok = ws.b_tok + size_t(b) * ws.cap_b;
  unsigned long long* a_key = ws.a_key + size_t(b) * ws.cap_a;
  __shared__ int max_ab[2][32];

  for (int i = tid; i < 32 * nW; i += blockDim.x) cnt[i] = 0;
  __syncthreads();

  const int seg = (n + 31) / 32;
  const int s0 = min(n, wp * seg), s1 = min(n, s0 + seg);

  // pass A: window id of every token, per-warp per-window counts
  for (int base = s0; base < s1; base += 32) {
    const int i = base + lane;
    const bool act = i < s1;
    const unsigned amask = __ballot_sync(0xffffffffu, act);
    if (act) {
      const int p = pos ? pos[i] : i;
      int w = window_of(g, p);
      const int prev = (i > 0) ? (pos ? pos[i - 1] : i - 1) : -1;
      if (w < 0 || p <= prev) { set_status(status, LIGHTKV_STATUS_POS_ORDER); if (w < 0) w = 0; }
      tok_win[i] = w;
      const unsigned peers = __match_any_sync(amask, w);
      if (lane == __ffs(peers) - 1) cnt[wp * nW + w] += (uint16_t)__popc(peers);
    }
    __syncwarp();
  }
  __syncthreads();

  // exclusive prefix over the 32 warp rows, window totals
  for (int w = tid; w < nW; w += blockDim.x) {
    int run = 0;
    for (int k = 0; k < 32; ++k) {
      const int c = cnt[k * nW + w];
      cnt[k * nW + w] = (uint16_t)run;
      run += c;
    }
    wsum[w] = run;
  }
  __syncthreads();

  // exclusive scans over windows: token offsets (wsum) and A-entry offsets (asum)
  if (wp == 0) {
    const int chunk = (nW + 31) / 32;
    const int lo = min(nW, lane * chunk), hi = min(nW, lo + chunk);
    int s = 0, sa = 0;
    for (int w = lo; w < hi; ++w) { s += wsum[w]; sa += (wsum[w] + 1 - g.src_par) >> 1; }
    int xs = s, xa = sa;
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, xs, o), ta = __shfl_up_sync(0xffffffffu, xa, o);
      if (lane >= o) { xs += t; xa += ta; }
    }
    xs -= s; xa -= sa;
    for (int w = lo; w < hi; ++w) {
      const int c = wsum[w];
      wsum[w] = xs; asum[w] = xa;
      xs += c; xa += (c + 1 - g.src_par) >> 1;
    }
    if (lane == 31) { wsum[nW] = xs; asum[nW] = xa; }
  }
  __syncthreads();
  // A sample whose A or B nodes do not fit the plan's capacities (a subset of the grid handed to a plan that was
  // built for full grids) keeps all of its tokens: its windows are published empty, so no later kernel finds an
  // entry, a tile or a window size for it, nothing is indexed past a row, and the status word says so.
  const bool over = asum[nW] > ws.cap_a || wsum[nW] - asum[nW] > ws.cap_b;
  if (over && tid == 0) set_status(status, LIGHTKV_STATUS_COUNT);
  for (int w = tid; w <= nW; w += blockDim.x) {
    ws.win_off[size_t(b) * (nW + 1) + w] = over ? 0 : wsum[w];
    ws.a_off[size_t(b) * (nW + 1) + w] = over ? 0 : asum[w];
  }
  {  // largest A and B side of any window -> tiling of the tensor-core FD kernel
    int ma = 0, mb = 0;
    for (int w = tid; w < nW; w += blockDim.x) {
      const int na = asum[w + 1] - asum[w];
      ma = max(ma, na);
      mb = max(mb, wsum[w + 1] - wsum[w] - na);
    }
    ma = __reduce_max_sync(0xffffffffu, ma);
    mb = __reduce_max_sync(0xffffffffu, mb);
    if (lane == 0) { max_ab[0][wp] = ma; max_ab[1][wp] = mb; }
    __syncthreads();
    if (wp == 0) {
      ma = __reduce_max_sync(0xffffffffu, max_ab[0][lane]);
      mb = __reduce_max_sync(0xffffffffu, max_ab[1][lane]);
      if (lane == 0) {
        FdTiling t;
        const int mm = max(ma, mb);                      // either side of a window (the destinations outnumber the
                                                         // sources by one per odd window in the reverse direction)
        if (mm <= kFdTile) {
          // as few windows per tile as still gives the batch about kFdTargetTiles tiles, at most 128 entries a side
          const int want = (nW * (int)gridDim.x + kFdTargetTiles - 1) / kFdTargetTiles;
          t.wpt = mm > 0 ? max(1, min(min(kFdTile / mm, nW), want)) : nW;
          t.blocks_a = 1; t.blocks_b = 1;
          const int rows = t.wpt * mm;
          t.passes = rows <= 32 ? 1 : (rows <= 64 ? 2 : 4);
        } else {
          t.wpt = 1;
          t.blocks_a = (ma + kFdTile - 1) / kFdTile; t.blocks_b = (mb + kFdTile - 1) / kFdTile;
          t.passes = 4;
        }
        t.n_tiles = (ma > 0 && mb > 0 && !over) ? ((nW + t.wpt - 1) / t.wpt) * t.blocks_a * t.blocks_b : 0;
        t.pad[0] = t.pad[1] = t.pad[2] = 0;
        ws.fd_tiling[b] = t;
      }
    }
  }

  // pass B: local rank, A / B entry lists
  for (int base = s0; base < s1; base += 32) {
    const int i = base + lane;
    const bool act = i < s1;
    const unsigned amask = __ballot_sync(0xffffffffu, act);
    if (act) {
      const int w = tok_win[i];
      const unsigned peers = __match_any_sync(amask, w);
      const int before = cnt[wp * nW + w];
      __syncwarp(amask);
      if (lane == __ffs(peers) - 1) cnt[wp * nW + w] = (uint16_t)(before + __popc(peers));
      __syncwarp(amask);
      const int l = before + __popc(peers & ((1u << lane) - 1u));
      tok_l[i] = l;
      if ((l & 1) != g.src_par) {
        const int e = (wsum[w] - asum[w]) + (l >> 1);
        if (e < ws.cap_b) b_tok[e] = i;
      } else {
        const int e = asum[w] + (l >> 1);
        if (e < ws.cap_a) { a_tok[e] = i; a_win[e] = w; a_key[e] = ~0ull; }
      }
    }
    __syncwarp();
  }
}

cudaError_t launch_window_build(const LayerLaunch& L) {
  const int nW = L.geo.n_windows;
  const size_t smem = ((size_t(32) * nW * 2 + 15) & ~size_t(15)) + size_t(2) * (nW + 1) * sizeof(int);
  const cudaError_t e = ensure_dynamic_smem(window_build_kernel, 200 * 1024);
  if (e != cudaSuccess) return e;
  return launch_kernel(window_build_kernel, L.batch, 1024, smem, L.stream, 1, L.geo, L.a->pos, L.a->n_vis, L.ws, L.a->status);
}

// =====================================================================================================
// FD + best partner, fp32 FMA path (Eq. "similarity", Step 2).
// One CTA per (sample, tile of 32 A entries).  The B entries of the windows the tile touches are
// visited in chunks of 64; G = X_A X_B^T accumulates in registers over k-chunks of 32 staged in smem,
// squared norms accumulate from the same staged tiles.  Every A row then scans the FD of its own
// window's B entries in ascending order (strict <, so ties go to the lowest B index).
// =====================================================================================================
constexpr int FD_TA = 32, FD_TB = 64, FD_KC = 32;

template <typename T>
__device__ inline void load4(const T* p, float (&f)[4]);
template <>
__device__ inline void load4<float>(const float* p, float (&f)[4]) {
  const float4 v = *reinterpret_cast<const float4*>(p);
  f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
template <>
__device__ inline void load4<__nv_bfloat16>(const __nv_bfloat16* p, float (&f)[4]) {
  const uint2 v = *reinterpret_cast<const uint2*>(p);
  f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
  f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
}

template <typename T>
__global__ void __launch_bounds__(256)
fd_simt_kernel(const T* __restrict__ hidden, int64_t batch_stride, int64_t row_stride, const int* __restrict__ seq_start,
               int vis_begin, int d, int metric, Workspace ws) {
  grid_dependency_sync();
  __shared__ float As[FD_TA][FD_KC + 1];
  __shared__ float Bs[FD_TB][FD_KC + 1];
  __shared__ float Gs[FD_TA][FD_TB + 1];
  __shared__ float a_ss[FD_TA], b_ss[FD_TB];
  __shared__ int a_row[FD_TA], b_row[FD_TB], a_lo[FD_TA], a_hi[FD_TA];

  const int b = blockIdx.y, tid = threadIdx.x;
  const int nW = ws.n_windows;
  const int* win_off = ws.win_off + size_t(b) * (nW + 1);
  const int* a_off = ws.a_off + size_t(b) * (nW + 1);
  const int* a_tok = ws.a_tok + size_t(b) * ws.cap_a;
  const int* a_win = ws.a_win + size_t(b) * ws.cap_a;
  const int* b_tok = ws.b_tok + size_t(b) * ws.cap_b;
  const int n_a = a_off[nW];
  const int e0 = blockIdx.x * FD_TA;
  if (e0 >= n_a) return;
  const int ne = min(FD_TA, n_a - e0);
  const T* x = hidden + size_t(b) * batch_stride + size_t((seq_start ? seq_start[b] : 0) + vis_begin) * row_stride;

  if (tid < FD_TA) {
    if (tid < ne) {
      const int w = a_win[e0 + tid];
      a_row[tid] = a_tok[e0 + tid];
      a_lo[tid] = win_off[w] - a_off[w];
      a_hi[tid] = win_off[w + 1] - a_off[w + 1];
    } else {
      a_row[tid] = -1; a_lo[tid] = 0; a_hi[tid] = 0;
    }
  }
  __syncthreads();
  const int bb0 = a_lo[0], bb1 = a_hi[ne - 1];

  const int tx = tid & 15, ty = tid >> 4;            // 4 B columns x 2 A rows per thread
  float best_f = 3.0e38f;                            // threads < ne: running minimum of their A row
  int best_e = -1;                                   // ... and the B entry that attains it
  float ssa = 0.f;                                   // threads < FD_TA: squared norm of A row tid

  for (int cb = bb0; cb < bb1; cb += FD_TB) {
    const int nb = min(FD_TB, bb1 - cb);
    if (tid < FD_TB) b_row[tid] = tid < nb ? b_tok[cb + tid] : -1;
    float acc[2][4] = {};
    float ssb = 0.f;                                 // threads 32..95: squared norm of B row tid-32
    const bool first = (cb == bb0);
    __syncthreads();
    for (int k0 = 0; k0 < d; k0 += FD_KC) {
      {  // stage A tile: 32 x 32, 4 elements per thread
        const int r = tid >> 3, c = (tid & 7) * 4;
        float f[4] = {0.f, 0.f, 0.f, 0.f};
        if (a_row[r] >= 0 && k0 + c < d) load4<T>(x + size_t(a_row[r]) * row_stride + k0 + c, f);
#pragma unroll
        for (int j = 0; j < 4; ++j) As[r][c + j] = f[j];
      }
#pragma unroll
      for (int half = 0; half < 2; ++half) {  // stage B tile: 64 x 32
        const int r = (tid >> 3) + half * 32, c = (tid & 7) * 4;
        float f[4] = {0.f, 0.f, 0.f, 0.f};
        if (b_row[r] >= 0 && k0 + c < d) load4<T>(x + size_t(b_row[r]) * row_stride + k0 + c, f);
#pragma unroll
        for (int j = 0; j < 4; ++j) Bs[r][c + j] = f[j];
      }
      __syncthreads();
#pragma unroll 8
      for (int kk = 0; kk < FD_KC; ++kk) {
        const float a0 = As[2 * ty][kk], a1 = As[2 * ty + 1][kk];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float bv = Bs[4 * tx + j][kk];
          acc[0][j] = fmaf(a0, bv, acc[0][j]);
          acc[1][j] = fmaf(a1, bv, acc[1][j]);
        }
      }
      if (first && tid < FD_TA) {
        for (int kk = 0; kk < FD_KC; ++kk) ssa = fmaf(As[tid][kk], As[tid][kk], ssa);
      } else if (tid >= 32 && tid < 32 + FD_TB) {
        for (int kk = 0; kk < FD_KC; ++kk) ssb = fmaf(Bs[tid - 32][kk], Bs[tid - 32][kk], ssb);
      }
      __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) Gs[2 * ty + i][4 * tx + j] = acc[i][j];
    if (first && tid < FD_TA) a_ss[tid] = ssa;
    if (tid >= 32 && tid < 32 + FD_TB) b_ss[tid - 32] = ssb;
    __syncthreads();
    if (tid < ne) {
      const int lo = max(a_lo[tid], cb), hi = min(a_hi[tid], cb + nb);
      const float na = sqrtf(a_ss[tid]);
      for (int e = lo; e < hi; ++e) {
        float fd;
        if (metric == LIGHTKV_FD_COSINE) {
          const float den = na * sqrtf(b_ss[e - cb]);
          fd = 1.0f - (den > 0.f ? Gs[tid][e - cb] / den : 0.f);
        } else {
          fd = fmaxf(fmaf(-2.0f, Gs[tid][e - cb], a_ss[tid] + b_ss[e - cb]), 0.f);   // |a|^2 + |b|^2 - 2 <a, b>
          if (metric == LIGHTKV_FD_L2) fd = sqrtf(fd);
        }
        if (fd < best_f) { best_f = fd; best_e = e; }
      }
    }
    __syncthreads();
  }
  if (tid < ne && best_e >= 0)
    ws.a_key[size_t(b) * ws.cap_a + e0 + tid] = ((unsigned long long)orderable(best_f) << 32) | (unsigned)best_e;
}

cudaError_t launch_fd_simt(const LayerLaunch& L) {
  const dim3 grid((L.ws.cap_a + FD_TA - 1) / FD_TA, L.batch);
  if (L.dtype == LIGHTKV_BF16)
    return launch_kernel(fd_simt_kernel<__nv_bfloat16>, grid, 256, 0, L.stream, 1,
                         static_cast<const __nv_bfloat16*>(L.a->hidden), L.a->hidden_batch_stride,
                         L.a->hidden_row_stride, L.a->seq_start, L.a->vis_begin, L.hidden, L.divergence, L.ws);
  return launch_kernel(fd_simt_kernel<float>, grid, 256, 0, L.stream, 1, static_cast<const float*>(L.a->hidden),
                       L.a->hidden_batch_stride, L.a->hidden_row_stride, L.a->seq_start, L.a->vis_begin, L.hidden,
                       L.divergence, L.ws);
}

// =====================================================================================================
// xi per head, fp32 FMA path (Eq. "attention-factor" with the causal softmax rows of Eq.
// "attention-matrix").  One CTA per (tile of 32 vision queries, head, sample).  Keys 0..s_i are visited
// in tiles of 64 with an online (running-maximum) softmax that carries two sums per row: all visible
// keys and the prompt keys J.  Output per head: sum_J / sum_all.  With a caller-supplied row
// log-sum-exp only the prompt keys are visited: sum_J exp(logit - lse).
// =====================================================================================================
constexpr int XI_TQ = 32, XI_TK = 64;

template <typename T>
struct XiSimtArgs {
  const T* q; int64_t q_bs, q_hs, q_rs;
  const T* k; int64_t k_bs, k_hs, k_rs;
  const float* lse; int64_t lse_bs, lse_hs;        // caller's row log-sum-exp (ATTN_LSE) or nullptr
  float* lse_out; int64_t lse_out_bs, lse_out_hs;  // receives the row log-sum-exp (ATTN_FULL) or nullptr
  const int* n_vis;
  const int* seq_start;                            // first row of each sample in q, k, lse, lse_out (packed batches) or nullptr
  int vis_begin, n_text_after, bidirectional;
  int n_q_heads, n_kv_heads, dh;
  TextSet text;
};

template <typename T>
__global__ void __launch_bounds__(256)
xi_simt_kernel(XiSimtArgs<T> a, Workspace ws) {
  grid_dependency_sync();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int dh = a.dh, ld = dh + 1;
  float* Qs = reinterpret_cast<float*>(smem_raw);       // [XI_TQ][ld]
  float* Ks = Qs + XI_TQ * ld;                          // [XI_TK][ld]
  float* Ss = Ks + XI_TK * ld;                          // [XI_TQ][XI_TK + 1]

  const int b = blockIdx.z, h = blockIdx.y, t0 = blockIdx.x * XI_TQ, tid = threadIdx.x;
  int n = a.n_vis ? min(a.n_vis[b], ws.cap_in) : ws.cap_in;
  if (t0 >= n) return;
  const int nq = min(XI_TQ, n - t0);
  const int hk = h / (a.n_q_heads / a.n_kv_heads);
  const int row0 = a.seq_start ? a.seq_start[b] : 0;
  const T* qh = a.q + size_t(b) * a.q_bs + size_t(h) * a.q_hs + size_t(row0) * a.q_rs;
  const T* kh = a.k + size_t(b) * a.k_bs + size_t(hk) * a.k_hs + size_t(row0) * a.k_rs;
  const float scale2 = 1.4426950408889634f / sqrtf((float)dh);      // logits in log2 units
  const int vis_begin = a.vis_begin;
  const int n_seq = vis_begin + n + a.n_text_after;                   // keys of this sample

  for (int idx = tid; idx < XI_TQ * (dh / 4); idx += blockDim.x) {
    const int r = idx / (dh / 4), c = (idx % (dh / 4)) * 4;
    float f[4] = {0.f, 0.f, 0.f, 0.f};
    if (r < nq) load4<T>(qh + size_t(vis_begin + t0 + r) * a.q_rs + c, f);
#pragma unroll
    for (int j = 0; j < 4; ++j) Qs[r * ld + c + j] = f[j];
  }

  const int tx = tid & 15, ty = tid >> 4;
  const int lane = tid & 31, wp = tid >> 5;             // softmax: warp wp owns rows 4*wp .. 4*wp+3
  float m_run[4], l_all[4], l_txt[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) { m_run[i] = -INFINITY; l_all[i] = 0.f; l_txt[i] = 0.f; }

  // last key any row of the tile may see: its own (causal) or the sample's last (bidirectional)
  const int s_last = a.bidirectional ? n_seq - 1 : vis_begin + t0 + nq - 1;
  const int key_lo = a.lse ? a.text.begin : 0;
  const int key_hi = a.lse ? min(a.text.end, s_last + 1) : s_last + 1;

  for (int j0 = key_lo; j0 < key_hi; j0 += XI_TK) {
    const int nk = min(XI_TK, key_hi - j0);
    __syncthreads();
    for (int idx = tid; idx < XI_TK * (dh / 4); idx += blockDim.x) {
      const int r = idx / (dh / 4), c = (idx % (dh / 4)) * 4;
      float f[4] = {0.f, 0.f, 0.f, 0.f};
      if (r < nk) load4<T>(kh + size_t(j0 + r) * a.k_rs + c, f);
#pragma unroll
      for (int j = 0; j < 4; ++j) Ks[r * ld + c + j] = f[j];
    }
    __syncthreads();
    float acc[2][4] = {};
    for (int kk = 0; kk < dh; ++kk) {
      const float a0 = Qs[(2 * ty) * ld + kk], a1 = Qs[(2 * ty + 1) * ld + kk];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float bv = Ks[(4 * tx + j) * ld + kk];
        acc[0][j] = fmaf(a0, bv, acc[0][j]);
        acc[1][j] = fmaf(a1, bv, acc[1][j]);
      }
    }
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) Ss[(2 * ty + i) * (XI_TK + 1) + 4 * tx + j] = acc[i][j] * scale2;
    __syncthreads();
    const unsigned long long tmask = a.text.mask64(j0);      // XI_TK = 64 columns
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = 4 * wp + i;
      if (r >= nq) continue;                            // warp-uniform
      const int s_i = vis_begin + t0 + r;
      const int last = a.bidirectional ? n_seq - 1 : s_i;
      float v[2];
      bool ok[2], txt[2];
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int j = j0 + lane + 32 * c;
        ok[c] = (lane + 32 * c < nk) && j <= last;
        txt[c] = ok[c] && ((tmask >> (lane + 32 * c)) & 1ull);
        v[c] = ok[c] ? Ss[r * (XI_TK + 1) + lane + 32 * c] : -INFINITY;
      }
      if (a.lse) {
        const float l2 = a.lse[size_t(b) * a.lse_bs + size_t(h) * a.lse_hs + row0 + s_i] * 1.4426950408889634f;
        float p = (txt[0] ? exp2f(v[0] - l2) : 0.f) + (txt[1] ? exp2f(v[1] - l2) : 0.f);
        for (int o = 16; o > 0; o >>= 1) p += __shfl_xor_sync(0xffffffffu, p, o);
        l_txt[i] += p;
        continue;
      }
      float mx = fmaxf(v[0], v[1]);
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_new = fmaxf(m_run[i], mx);          // finite: key 0 is visible to every query
      const float p0 = ok[0] ? exp2f(v[0] - m_new) : 0.f, p1 = ok[1] ? exp2f(v[1] - m_new) : 0.f;
      float sa = p0 + p1, st = (txt[0] ? p0 : 0.f) + (txt[1] ? p1 : 0.f);
      for (int o = 16; o > 0; o >>= 1) {
        sa += __shfl_xor_sync(0xffffffffu, sa, o);
        st += __shfl_xor_sync(0xffffffffu, st, o);
      }
      const float resc = exp2f(m_run[i] - m_new);       // 0 on the first tile (m_run = -inf)
      l_all[i] = l_all[i] * resc + sa;
      l_txt[i] = l_txt[i] * resc + st;
      m_run[i] = m_new;
    }
  }
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = 4 * wp + i;
      if (r < nq) {
        ws.xi_h[(size_t(b) * a.n_q_heads + h) * ws.cap_in + t0 + r] = a.lse ? l_txt[i] : l_txt[i] / l_all[i];
        if (a.lse_out)
          a.lse_out[size_t(b) * a.lse_out_bs + size_t(h) * a.lse_out_hs + row0 + vis_begin + t0 + r] =
              (m_run[i] + log2f(l_all[i])) * 0.6931471805599453f;
      }
    }
  }
}

template <typename T>
static cudaError_t launch_xi_simt_t(const LayerLaunch& L) {
  const lightkv_layer_args_t* a = L.a;
  const int dh = L.head_dim;
  const size_t smem = (size_t(XI_TQ + XI_TK) * (dh + 1) + size_t(XI_TQ) * (XI_TK + 1)) * sizeof(float);
  const dim3 grid((L.ws.cap_in + XI_TQ - 1) / XI_TQ, L.n_q_heads, L.batch);
  XiSimtArgs<T> x;
  x.q = static_cast<const T*>(a->q); x.q_bs = a->q_batch_stride; x.q_hs = a->q_head_stride; x.q_rs = a->q_row_stride;
  x.k = static_cast<const T*>(a->k); x.k_bs = a->k_batch_stride; x.k_hs = a->k_head_stride; x.k_rs = a->k_row_stride;
  x.lse = L.xi_mode == LIGHTKV_XI_ATTN_LSE ? a->lse : nullptr; x.lse_bs = a->lse_batch_stride; x.lse_hs = a->lse_head_stride;
  x.lse_out = L.xi_mode == LIGHTKV_XI_ATTN_FULL ? a->lse_out : nullptr;
  x.lse_out_bs = a->lse_out_batch_stride; x.lse_out_hs = a->lse_out_head_stride;
  x.n_vis = a->n_vis; x.seq_start = a->seq_start;
  x.vis_begin = a->vis_begin; x.n_text_after = a->n_text_after; x.bidirectional = a->bidirectional;
  x.n_q_heads = L.n_q_heads; x.n_kv_heads = L.n_kv_heads; x.dh = dh; x.text = L.text;
  const cudaError_t e = ensure_dynamic_smem(xi_simt_kernel<T>, 160 * 1024);
  if (e != cudaSuccess) return e;
  return launch_kernel(xi_simt_kernel<T>, grid, 256, smem, L.stream, 1, x, L.ws);
}

cudaError_t launch_xi_simt(const LayerLaunch& L) {
  return L.dtype == LIGHTKV_BF16 ? launch_xi_simt_t<__nv_bfloat16>(L) : launch_xi_simt_t<float>(L);
}

// =====================================================================================================
// Selection + merge map (Steps 2-5).  One cluster of 1-8 CTAs per sample (about a token per thread); every
// CTA keeps a contiguous range of the sample's tokens through all phases, phases that read what other
// threads wrote are separated by cluster barriers, prefix sums cross the cluster through distributed shared
// memory.
//   1  xi = fixed-order sum over heads (or given / uniform); every source token (local rank parity src_par): r =
//      removal_count(n_w), selected iff it is among the r entries of its window with the smallest
//      (FD, index) (rank by counting 32-bit keys; skipped when r = |A|); a selected token takes its best B
//   2  survivors (all B, unselected A) get consecutive output slots in storage (= position) order: dst,
//      pos_out, and a group of one member each
//   3  a merged token joins its partner's group (integer atomic on the size); its place in the group is
//      the number of earlier entries of its window with the same partner
//   4  group sizes -> grp_off (scan)
//   5  grp_src: the survivor first, then its merged A tokens in entry order
//   6  weights xi_i / sum over the group, the sum taken in that fixed order
// =====================================================================================================
struct SelectArgs {
  int n_q_heads, xi_mode, cap_out, src_par;
  double keep;
  const int* n_vis;
  const int* pos;
  const float* xi_in;
  int* n_vis_out;
  int* pos_out;
  int* dst;
  float* weight;
  int* grp_off;
  int* grp_src;
  float* xi_out;
  uint32_t* status;
};

// exclusive scan of one value per thread across the CTA; returns the exclusive prefix, total in *total
__device__ inline int block_exclusive_scan(int v, int* warp_sums /* [33] smem */, int* total) {
  const int lane = threadIdx.x & 31, wp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  int x = v;
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += t;
  }
  __syncthreads();                       // warp_sums may still be read from the previous call
  if (lane == 31) warp_sums[wp] = x;
  __syncthreads();
  if (wp == 0) {
    int s = lane < nwarps ? warp_sums[lane] : 0;
    const int own = s;
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, s, o);
      if (lane >= o) s += t;
    }
    warp_sums[lane] = s - own;
    if (lane == 31) warp_sums[32] = s;
  }
  __syncthreads();
  *total = warp_sums[32];
  return warp_sums[wp] + x - v;
}

// CLUSTER = false: one CTA per sample, plain launch, block barriers only.
template <bool CLUSTER>
__global__ void __launch_bounds__(1024) select_map_kernel(Workspace ws, SelectArgs a) {
  grid_dependency_sync();
  __shared__ int warp_sums[33];
  __shared__ int cta_total[2];                  // survivors / group members counted by this CTA
  const int cs = CLUSTER ? (int)tc::cluster_nctarank() : 1, rank = CLUSTER ? (int)tc::cluster_ctarank() : 0;
  auto sync_all = [&]() { if (CLUSTER) tc::cluster_sync(); else __syncthreads(); };
  const int b = blockIdx.x / cs, tid = threadIdx.x, nthr = blockDim.x;
  const int gtid = rank * nthr + tid;                        // thread index inside the cluster
  const int nW = ws.n_windows;
  int n = a.n_vis ? min(a.n_vis[b], ws.cap_in) : ws.cap_in;
  if (n < 0) n = 0;
  const int* win_off = ws.win_off + size_t(b) * (nW + 1);
  const int* a_off = ws.a_off + size_t(b) * (nW + 1);
  const int* tok_win = ws.tok_win + size_t(b) * ws.cap_in;
  const int* tok_l = ws.tok_l + size_t(b) * ws.cap_in;
  const unsigned long long* a_key = ws.a_key + size_t(b) * ws.cap_a;
  const int* b_tok = ws.b_tok + size_t(b) * ws.cap_b;
  float* xi = ws.xi + size_t(b) * ws.cap_in;
  int* partner = ws.partner + size_t(b) * ws.cap_in;
  int* slot = ws.slot + size_t(b) * ws.cap_in;
  int* a_partner = ws.a_partner + size_t(b) * ws.cap_a;
  const int* pos = a.pos ? a.pos + size_t(b) * ws.cap_in : nullptr;
  int* dst = a.dst + size_t(b) * ws.cap_in;
  float* weight = a.weight + size_t(b) * ws.cap_in;
  int* grp_off = a.grp_off + size_t(b) * (a.cap_out + 1);
  int* grp_src = a.grp_src + size_t(b) * ws.cap_in;
  int* pos_out = a.pos_out + size_t(b) * a.cap_out;

  // Every CTA of the cluster owns a contiguous range of the sample's tokens; a thread keeps the same tokens
  // in every phase, so what it wrote for a token it may read back without a barrier.
  const int chunk = (n + cs - 1) / cs, lo = min(n, rank * chunk), hi = min(n, lo + chunk);

  // Exclusive scan of `value(i)` over the cluster: CTA `rank` owns [s_lo, s_hi) (at most s_chunk long, the
  // same bound in every CTA), counts it, learns the ranges before it through distributed shared memory,
  // then scans it.  emit(i, prefix) is called for every i; returns the grand total.
  auto cluster_scan = [&](int s_lo, int s_hi, int s_chunk, int which, auto value, auto emit) {
    int before = 0, grand = 0;
    auto exchange = [&](int mine) {
      if (tid == 0) cta_total[which] = mine;
      tc::cluster_sync();
      for (int j = 0; j < cs; ++j) {
        const int t = (int)tc::ld_cluster_u32(tc::map_to_cta(tc::smem_u32(&cta_total[which]), j));
        if (j < rank) before += t;
        grand += t;
      }
    };
    if (s_chunk <= nthr) {                              // one value per thread: a single pass
      const int i = s_lo + tid;
      int total;
      const int ex = block_exclusive_scan(i < s_hi ? value(i) : 0, warp_sums, &total);
      if (CLUSTER) exchange(total); else grand = total;
      if (i < s_hi) emit(i, before + ex);
      return grand;
    }
    if (CLUSTER) {
      int mine = 0;
      for (int base = s_lo; base < s_hi; base += nthr) {
        const int i = base + tid;
        int total;
        block_exclusive_scan(i < s_hi ? value(i) : 0, warp_sums, &total);
        mine += total;
      }
      exchange(mine);
    }
    int carry = before;
    for (int base = s_lo; base < s_hi; base += nthr) {
      const int i = base + tid;
      int total;
      const int ex = block_exclusive_scan(i < s_hi ? value(i) : 0, warp_sums, &total);
      if (i < s_hi) emit(i, carry + ex);
      carry += total;
    }
    return CLUSTER ? grand : carry;
  };

  // phase 1: xi of every token; every A token (even local rank, entry a_off[w] + l / 2) decides whether it is
  // among the r lowest-FD entries of its window and, if so, takes the partner FD found for it
  const uint32_t* key_word = reinterpret_cast<const uint32_t*>(a_key);   // [2e]: best B entry, [2e + 1]: orderable FD
  for (int i = lo + tid; i < hi; i += nthr) {
    float v;
    if (a.xi_mode == LIGHTKV_XI_GIVEN) v = a.xi_in[size_t(b) * ws.cap_in + i];
    else if (a.xi_mode == LIGHTKV_XI_UNIFORM) v = 1.0f;
    else {
      v = 0.f;
#pragma unroll 8
      for (int h = 0; h < a.n_q_heads; ++h) v += ws.xi_h[(size_t(b) * a.n_q_heads + h) * ws.cap_in + i];
    }
    xi[i] = v;
    if (a.xi_out) a.xi_out[size_t(b) * ws.cap_in + i] = v;
    int p = -1;
    const int l = tok_l[i];
    if ((l & 1) == a.src_par) {                        // a source node
      const int w = tok_win[i];
      const int e_lo = a_off[w], e_hi = a_off[w + 1], e = e_lo + (l >> 1);
      if (e < ws.cap_a) {
        const int r = removal_count(win_off[w + 1] - win_off[w], a.keep, a.src_par);
        bool sel;
        if (r <= 0) sel = false;
        else if (r >= e_hi - e_lo) sel = true;
        else {
          // rank in the order (lowest FD, A entry index): entries before e win ties, entries after e lose them
          const uint32_t mine = key_word[2 * e + 1];
          int rk = 0;
          for (int e2 = e_lo; e2 < e; ++e2) rk += (key_word[2 * e2 + 1] <= mine);
          for (int e2 = e + 1; e2 < e_hi; ++e2) rk += (key_word[2 * e2 + 1] < mine);
          sel = rk < r;
        }
        const uint32_t best_e = key_word[2 * e];
        p = (sel && best_e != 0xffffffffu) ? b_tok[best_e] : -1;
        a_partner[e] = p;                              // entry-indexed copy: phase 3 counts over it in order
      }
    }
    partner[i] = p;
  }

  // phase 2: output slot of every surviving token (its own tokens: no barrier needed before); the survivor
  // opens its group with one member
  const int survivors = cluster_scan(lo, hi, chunk, 0, [&](int i) { return partner[i] < 0 ? 1 : 0; },
                                     [&](int i, int prefix) {
                                       if (partner[i] >= 0) return;
                                       slot[i] = prefix;
                                       dst[i] = prefix;
                                       if (prefix >= a.cap_out) return;
                                       pos_out[prefix] = pos ? pos[i] : i;
                                       grp_off[prefix] = 1;
                                     });
  const int n_out = min(survivors, a.cap_out);
  if (gtid == 0) {
    a.n_vis_out[b] = n_out;
    if (survivors > a.cap_out) set_status(a.status, LIGHTKV_STATUS_COUNT);
  }
  sync_all();

  // phase 3: a merged token joins the group of its partner; its place in the group is the number of earlier
  // entries of its window with the same partner (kept in slot[], which a merged token does not use otherwise)
  for (int i = lo + tid; i < hi; i += nthr) {
    const int p = partner[i];
    if (p < 0) continue;
    const int o = slot[p];
    dst[i] = o;
    const int e_lo = a_off[tok_win[i]], e = e_lo + (tok_l[i] >> 1);
    int rk = 0;
    for (int e2 = e_lo; e2 < e; ++e2) rk += (a_partner[e2] == p);
    slot[i] = rk;
    if (o < a.cap_out) atomicAdd(&grp_off[o], 1);
  }
  sync_all();

  // phase 4: group sizes -> group offsets
  const int chunk_o = (n_out + cs - 1) / cs, lo_o = min(n_out, rank * chunk_o), hi_o = min(n_out, lo_o + chunk_o);
  const int members = cluster_scan(lo_o, hi_o, chunk_o, 1, [&](int o) { return grp_off[o]; },
                                   [&](int o, int prefix) { grp_off[o] = prefix; });
  if (gtid == 0) grp_off[n_out] = members;
  sync_all();

  // phase 5: member lists, the surviving token first, then the merged ones in entry order
  for (int i = lo + tid; i < hi; i += nthr) {
    const int o = dst[i];
    if (o >= a.cap_out) continue;
    grp_src[grp_off[o] + (partner[i] < 0 ? 0 : 1 + slot[i])] = i;
  }
  sync_all();

  // phase 6: weights xi_i / (sum of xi over the group), the sum taken in member order
  for (int i = lo + tid; i < hi; i += nthr) {
    if (partner[i] >= 0) continue;
    const int o = slot[i];
    if (o >= a.cap_out) continue;
    const int g0 = grp_off[o], g1 = grp_off[o + 1];
    float den = 0.f;
    for (int c = g0; c < g1; ++c) den += xi[grp_src[c]];
    if (den >= 1e-30f) {
      for (int c = g0; c < g1; ++c) { const int t = grp_src[c]; weight[t] = xi[t] / den; }
    } else {
      set_status(a.status, LIGHTKV_STATUS_ZERO_WEIGHT);
      for (int c = g0; c < g1; ++c) weight[grp_src[c]] = 1.0f / (float)(g1 - g0);
    }
  }
}

cudaError_t launch_select_map(const LayerLaunch& L) {
  const lightkv_layer_args_t* a = L.a;
  SelectArgs s;
  s.n_q_heads = L.n_q_heads; s.xi_mode = L.xi_mode; s.cap_out = L.ws.cap_out; s.keep = L.keep;
  s.src_par = L.geo.src_par;
  s.n_vis = a->n_vis; s.pos = a->pos; s.xi_in = a->xi; s.n_vis_out = a->n_vis_out; s.pos_out = a->pos_out;
  s.dst = a->dst; s.weight = a->weight; s.grp_off = a->grp_off; s.grp_src = a->grp_src;
  s.xi_out = a->xi_out; s.status = a->status;
  // one cluster per sample: 1, 2, 4 or 8 CTAs of 1024 threads, about one token per thread
  const int cs = L.ws.cap_in <= 1024 ? 1 : (L.ws.cap_in <= 2048 ? 2 : (L.ws.cap_in <= 4096 ? 4 : 8));
  if (cs == 1) return launch_kernel(select_map_kernel<false>, L.batch, 1024, 0, L.stream, 1, L.ws, s);
  return launch_kernel(select_map_kernel<true>, L.batch * cs, 1024, 0, L.stream, cs, L.ws, s);
}

// =====================================================================================================
// Weighted merge of the hidden states (Eq. "message-passing", Steps 3-5): one CTA per output row.
// Row o of the vision block is sum over its group of weight_i * x_i in fp32, rounded once to the
// storage type; a group of one has weight exactly 1 and is therefore copied bit-exactly.  Text rows
// before / after the vision block are copied.  Pure 16-byte streaming loads and stores.
// =====================================================================================================
template <typename T>
__global__ void __launch_bounds__(256)
merge_rows_kernel(const T* __restrict__ src, int64_t src_bs, int64_t src_rs,
                  T* __restrict__ out, int64_t out_bs, int64_t out_rs,
                  int d, int vis_begin, int n_text_after, int cap_in, int cap_out,
                  const int* __restrict__ n_vis, const int* __restrict__ n_vis_out,
                  const int* __restrict__ grp_off, const int* __restrict__ grp_src,
                  const float* __restrict__ weight, const int* __restrict__ seq_start,
                  const int* __restrict__ seq_start_out) {
  grid_dependency_sync();
  constexpr int V = Vec<T>::n;
  const int b = blockIdx.y, row = blockIdx.x;
  const int n_in = n_vis ? min(n_vis[b], cap_in) : cap_in;
  const int n_out = n_vis_out[b];
  if (row >= vis_begin + n_out + n_text_after) return;
  const T* sb = src + size_t(b) * src_bs + size_t(seq_start ? seq_start[b] : 0) * src_rs;
  T* orow = out + size_t(b) * out_bs + size_t((seq_start_out ? seq_start_out[b] : 0) + row) * out_rs;
  const int chunks = d / V;
  if (row < vis_begin || row >= vis_begin + n_out) {
    const T* srow = sb + size_t(row < vis_begin ? row : row - n_out + n_in) * src_rs;
    for (int c0 = threadIdx.x; c0 < chunks; c0 += 2 * blockDim.x) {
      const int c1 = c0 + blockDim.x;
      const uint4 a0 = ld_stream16(srow + c0 * V);
      if (c1 < chunks) {
        const uint4 a1 = ld_stream16(srow + c1 * V);
        st_stream16(orow + c1 * V, a1);
      }
      st_stream16(orow + c0 * V, a0);
    }
    return;
  }
  const int o = row - vis_begin;
  const int* go = grp_off + size_t(b) * (cap_out + 1);
  const int g0 = go[o], g1 = go[o + 1];
  const int* gs = grp_src + size_t(b) * cap_in;
  const float* wt = weight + size_t(b) * cap_in;
  const T* vis = sb + size_t(vis_begin) * src_rs;
  // two 16-byte chunks per thread and two members at a time: four loads in flight whatever the group's size
  for (int c0 = threadIdx.x; c0 < chunks; c0 += 2 * blockDim.x) {
    const int c1 = c0 + blockDim.x;
    const bool two = c1 < chunks;
    float acc0[V], acc1[V];
#pragma unroll
    for (int j = 0; j < V; ++j) { acc0[j] = 0.f; acc1[j] = 0.f; }
    for (int g = g0; g < g1; g += 2) {
      uint4 va[2], vb[2];
      float wv[2];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        if (g + u < g1) {
          const int i = gs[g + u];
          wv[u] = wt[i];
          const T* r = vis + size_t(i) * src_rs;
          va[u] = ld_stream16(r + c0 * V);
          if (two) vb[u] = ld_stream16(r + c1 * V);
        }
      }
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        if (g + u < g1) {
          float f[V];
          unpack16(va[u], f, T());
#pragma unroll
          for (int j = 0; j < V; ++j) acc0[j] = fmaf(wv[u], f[j], acc0[j]);
          if (two) {
            unpack16(vb[u], f, T());
#pragma unroll
            for (int j = 0; j < V; ++j) acc1[j] = fmaf(wv[u], f[j], acc1[j]);
          }
        }
      }
    }
    st_stream16(orow + c0 * V, pack16(acc0, T()));
    if (two) st_stream16(orow + c1 * V, pack16(acc1, T()));
  }
}

cudaError_t launch_merge_rows(const LayerLaunch& L) {
  const lightkv_layer_args_t* a = L.a;
  const int rows = a->vis_begin + L.ws.cap_out + a->n_text_after;
  const dim3 grid(rows, L.batch);
  if (L.dtype == LIGHTKV_BF16)
    return launch_kernel(merge_rows_kernel<__nv_bfloat16>, grid, 256, 0, L.stream, 1,
        static_cast<const __nv_bfloat16*>(a->hidden), a->hidden_batch_stride, a->hidden_row_stride,
        static_cast<__nv_bfloat16*>(a->hidden_out), a->hidden_out_batch_stride, a->hidden_out_row_stride,
        L.hidden, a->vis_begin, a->n_text_after, L.ws.cap_in, L.ws.cap_out, a->n_vis, a->n_vis_out,
        a->grp_off, a->grp_src, a->weight, a->seq_start, a->seq_start_out);
  return launch_kernel(merge_rows_kernel<float>, grid, 256, 0, L.stream, 1,
        static_cast<const float*>(a->hidden), a->hidden_batch_stride, a->hidden_row_stride,
        static_cast<float*>(a->hidden_out), a->hidden_out_batch_stride, a->hidden_out_row_stride,
        L.hidden, a->vis_begin, a->n_text_after, L.ws.cap_in, L.ws.cap_out, a->n_vis, a->n_vis_out,
        a->grp_off, a->grp_src, a->weight, a->seq_start, a->seq_start_out);
}

// =====================================================================================================
// K/V merge-compaction (the cache of a layer shrinks together with its tokens: appendix "Method overview").
// The stage's merge map is applied per KV head; contiguous (strided) or paged (block-table) addressing
// on either side.  One CTA per output token, five CTAs per SM; every thread resolves the token's group
// itself (uniform, cached loads) and works on two 16-byte units and two group members at a time, i.e.
// four loads in flight whatever the group's size (four units on the copy path).  Groups of one are
// copied; larger groups are summed in fp32 in member order.
// =====================================================================================================
struct KvAddr {
  int64_t batch_stride, head_stride, row_stride, page_stride;
  const int* table;       // nullptr = contiguous
  int page_size, max_blocks;
  const int* seq_start;   // first token of each sample (packed caches) or nullptr
  __device__ inline int64_t token(int b, int n) const {
    if (seq_start) n += seq_start[b];
    if (!table) return int64_t(b) * batch_stride + int64_t(n) * row_stride;
    const int page = table[size_t(b) * max_blocks + n / page_size];
    return int64_t(page) * page_stride + int64_t(n % page_size) * row_stride;
  }
};

constexpr int KV_THREADS = 256;

// floor(n / d) for n, d < 65536 with m = ceil(2^32 / d): one multiply instead of a division
__device__ inline int div_magic(int n, unsigned m) { return (int)__umulhi((unsigned)n, m); }

template <typename T>
__global__ void __launch_bounds__(KV_THREADS, sizeof(T) == 2 ? 5 : 4)
kv_compact_kernel(const T* __restrict__ k_src, const T* __restrict__ v_src, T* __restrict__ k_dst,
                  T* __restrict__ v_dst, KvAddr sa, KvAddr da, int n_kv_heads, int dh, int vis_begin,
                  int n_text_after, int cap_in, int cap_out, int gather, int merge_at_survivor, unsigned magic_ch,
                  const int* __restrict__ n_vis, const int* __restrict__ n_vis_out,
                  const int* __restrict__ grp_off, const int* __restrict__ grp_src,
                  const float* __restrict__ weight) {
  grid_dependency_sync();
  constexpr int V = Vec<T>::n;
  const int b = blockIdx.y, row = blockIdx.x;
  const int n_in = n_vis ? min(n_vis[b], cap_in) : cap_in;
  const int n_out = n_vis_out[b];
  if (row >= vis_begin + n_out + n_text_after) return;
  const int ch = dh / V, per_kv = n_kv_heads * ch, units = 2 * per_kv;
  int64_t d_tok = da.token(b, row);
  const bool text = row < vis_begin || row >= vis_begin + n_out;
  const int* gs = grp_src + size_t(b) * cap_in;
  const float* wt = weight + size_t(b) * cap_in;
  int g0 = 0, g1 = 1;
  if (!text) {
    const int* go = grp_off + size_t(b) * (cap_out + 1);
    g0 = go[row - vis_begin];
    g1 = gather ? g0 + 1 : go[row - vis_begin + 1];
  }
  if (merge_at_survivor) {
    // first phase of the in-place form: a merged group is written over its surviving token's own row (no other
    // group reads that row); rows that are only moved wait for the second phase
    if (text || g1 - g0 == 1) return;
    d_tok = da.token(b, vis_begin + gs[g0]);
  }
  if (text || g1 - g0 == 1) {                                       // copy: text, lone survivor, gather mode
    const int64_t s_tok = text ? sa.token(b, row < vis_begin ? row : row - n_out + n_in)
                               : sa.token(b, vis_begin + gs[g0]);
    for (int u0 = threadIdx.x; u0 < units; u0 += 4 * blockDim.x) {   // four units' loads in flight per thread
      uint4 v[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int u = u0 + q * blockDim.x;
        if (u < units) {
          const int kv = u >= per_kv ? 1 : 0, rem = u - kv * per_kv, h = div_magic(rem, magic_ch), c = rem - h * ch;
          v[q] = ld_stream16((kv ? v_src : k_src) + s_tok + int64_t(h) * sa.head_stride + c * V);
        }
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int u = u0 + q * blockDim.x;
        if (u < units) {
          const int kv = u >= per_kv ? 1 : 0, rem = u - kv * per_kv, h = div_magic(rem, magic_ch), c = rem - h * ch;
          st_stream16((kv ? v_dst : k_dst) + d_tok + int64_t(h) * da.head_stride + c * V, v[q]);
        }
      }
    }
    return;
  }
  // merge: two units per thread and two members at a time, i.e. four loads in flight whatever the group's size
  for (int u0 = threadIdx.x; u0 < units; u0 += 2 * blockDim.x) {
    const int u1 = u0 + blockDim.x;
    const bool two = u1 < units;
    const int kv0 = u0 >= per_kv ? 1 : 0, rem0 = u0 - kv0 * per_kv, h0 = div_magic(rem0, magic_ch), c0 = rem0 - h0 * ch;
    const int ub = two ? u1 : u0;
    const int kv1 = ub >= per_kv ? 1 : 0, rem1 = ub - kv1 * per_kv, h1 = div_magic(rem1, magic_ch), c1 = rem1 - h1 * ch;
    const T* sp0 = (kv0 ? v_src : k_src) + int64_t(h0) * sa.head_stride + c0 * V;
    const T* sp1 = (kv1 ? v_src : k_src) + int64_t(h1) * sa.head_stride + c1 * V;
    float acc0[V], acc1[V];
#pragma unroll
    for (int j = 0; j < V; ++j) { acc0[j] = 0.f; acc1[j] = 0.f; }
    for (int g = g0; g < g1; g += 2) {
      uint4 va[2], vb[2];
      float wv[2];
#pragma unroll
      for (int m = 0; m < 2; ++m) {
        if (g + m < g1) {
          const int i = gs[g + m];
          wv[m] = wt[i];
          const int64_t tok = sa.token(b, vis_begin + i);
          va[m] = ld_stream16(sp0 + tok);
          if (two) vb[m] = ld_stream16(sp1 + tok);
        }
      }
#pragma unroll
      for (int m = 0; m < 2; ++m) {
        if (g + m < g1) {
          float f[V];
          unpack16(va[m], f, T());
#pragma unroll
          for (int j = 0; j < V; ++j) acc0[j] = fmaf(wv[m], f[j], acc0[j]);
          if (two) {
            unpack16(vb[m], f, T());
#pragma unroll
            for (int j = 0; j < V; ++j) acc1[j] = fmaf(wv[m], f[j], acc1[j]);
          }
        }
      }
    }
    st_stream16((kv0 ? v_dst : k_dst) + d_tok + int64_t(h0) * da.head_stride + c0 * V, pack16(acc0, T()));
    if (two) st_stream16((kv1 ? v_dst : k_dst) + d_tok + int64_t(h1) * da.head_stride + c1 * V, pack16(acc1, T()));
  }
}

// =====================================================================================================
// Second phase of the in-place form: every output row moves from its surviving token's row (which holds the
// merged group after the first phase) to its slot.  A slot never lies behind its source (o <= i), so rows only
// move towards the front.  One CTA owns a plane -- one (sample, K or V, head, column part) -- and sweeps its
// output rows in ascending chunks: the sources of a chunk are gathered into shared memory, the CTA
// synchronises, the chunk is stored.  The sources of chunk k + 1 lie at or behind its first slot, i.e. behind
// everything chunk k writes, so its gather is issued before chunk k is stored; and a chunk's own sources are in
// shared memory before any of its slots is written.  Rows before the vision block do not move.
// =====================================================================================================
constexpr int KVM_THREADS = 256, KVM_CHUNK_BYTES = 40 * 1024;

template <typename T>
__global__ void __launch_bounds__(KVM_THREADS)
kv_move_kernel(T* __restrict__ k_buf, T* __restrict__ v_buf, KvAddr ad, int n_kv_heads, int dh, int parts,
               int vis_begin, int n_text_after, int cap_in, const int* __restrict__ n_vis,
               const int* __restrict__ n_vis_out, const int* __restrict__ grp_off, const int* __restrict__ grp_src,
               int cap_out) {
  grid_dependency_sync();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int V = Vec<T>::n;
  int plane = blockIdx.x;
  const int part = plane % parts; plane /= parts;
  const int h = plane % n_kv_heads; plane /= n_kv_heads;
  const int kv = plane & 1, b = plane >> 1;
  const int n_in = n_vis ? min(n_vis[b], cap_in) : cap_in;
  const int n_out = n_vis_out[b];
  if (n_out >= n_in) return;                               // nothing was merged away: every row is where it belongs
  T* buf = (kv ? v_buf : k_buf) + int64_t(h) * ad.head_stride;
  const int ch_all = dh / V, ch0 = part * ch_all / parts, ch = (part + 1) * ch_all / parts - ch0;   // 16-byte pieces of this plane
  const int rows_per_chunk = KVM_CHUNK_BYTES / (ch * 16);
  const int* go = grp_off + size_t(b) * (cap_out + 1);
  const int* gs = grp_src + size_t(b) * cap_in;
  const int row_end = vis_begin + n_out + n_text_after;
  const uint32_t sbase = tc::smem_u32(smem_raw);
  auto source = [&](int row) {                            // row of the buffer that holds output row `row`
    return row < vis_begin + n_out ? vis_begin + gs[go[row - vis_begin]] : row - n_out + n_in;
  };
  auto gather = [&](int r0, uint32_t sm) {                // output rows r0 .. of one chunk -> shared memory
    const int nr = min(rows_per_chunk, row_end - r0);
    for (int idx = threadIdx.x; idx < nr * ch; idx += blockDim.x) {
      const int rr = idx / ch, c = idx - rr * ch;
      tc::cp_async16(sm + uint32_t(idx) * 16, buf + ad.token(b, source(r0 + rr)) + (ch0 + c) * V, 16);
    }
  };
  int r0 = vis_begin, k = 0;
  gather(r0, sbase);
  tc::cp_async_commit();
  for (; r0 < row_end; r0 += rows_per_chunk, ++k) {
    const int next = r0 + rows_per_chunk;
    if (next < row_end) gather(next, sbase + ((k + 1) & 1) * KVM_CHUNK_BYTES);
    tc::cp_async_commit();
    tc::cp_async_wait<1>();                               // this thread's pieces of chunk k have landed
    __syncthreads();                                      // ... and everybody else's: all sources of chunk k are on chip
    const int nr = min(rows_per_chunk, row_end - r0);
    const unsigned char* sm = smem_raw + (k & 1) * KVM_CHUNK_BYTES;
    for (int idx = threadIdx.x; idx < nr * ch; idx += blockDim.x) {
      const int rr = idx / ch, c = idx - rr * ch;
      const uint4 v = *reinterpret_cast<const uint4*>(sm + size_t(idx) * 16);
      st_stream16(buf + ad.token(b, r0 + rr) + (ch0 + c) * V, v);
    }
    __syncthreads();                                      // the buffer may be refilled two chunks on
  }
  tc::cp_async_wait<0>();
}

cudaError_t launch_kv_compact(const KvLaunch& K) {
  const lightkv_kv_args_t* a = K.a;
  KvAddr sa{a->src_batch_stride, a->src_head_stride, a->src_row_stride, a->src_page_stride,
            a->page_size > 0 ? a->src_block_table : nullptr, a->page_size, a->max_blocks, a->src_seq_start};
  KvAddr da{a->dst_batch_stride, a->dst_head_stride, a->dst_row_stride, a->dst_page_stride,
            a->page_size > 0 ? a->dst_block_table : nullptr, a->page_size, a->max_blocks, a->dst_seq_start};
  const int ch_host = K.head_dim * (K.dtype == LIGHTKV_BF16 ? 2 : 4) / 16;
  if (2 * K.n_kv_heads * ch_host >= 65536) return cudaErrorInvalidValue;      // range of the unit decode
  const unsigned magic_ch = (unsigned)(((1ull << 32) + ch_host - 1) / ch_host);
  const dim3 grid(a->vis_begin + K.cap_out + a->n_text_after, K.batch);
  const int units = 2 * K.n_kv_heads * ch_host;
  // two units per thread (both in flight); narrow caches (GQA) get narrow CTAs
  const int threads = std::min(KV_THREADS, ((units + 1) / 2 + 31) / 32 * 32);
  const int gather = a->mode == LIGHTKV_KV_GATHER;
  const bool in_place = a->k_src == a->k_dst;             // (the API checked that V and the addressing agree)
  auto run = [&](auto tag) -> cudaError_t {
    using T = decltype(tag);
    cudaError_t e = cudaSuccess;
    if (!(in_place && gather))                            // in place, gather mode has nothing to merge
      e = launch_kernel(kv_compact_kernel<T>, grid, threads, 0, K.stream, 1,
          static_cast<const T*>(a->k_src), static_cast<const T*>(a->v_src), static_cast<T*>(a->k_dst),
          static_cast<T*>(a->v_dst), sa, da, K.n_kv_heads, K.head_dim, a->vis_begin, a->n_text_after, K.cap_in,
          K.cap_out, gather, in_place ? 1 : 0, magic_ch, a->n_vis, a->n_vis_out, a->grp_off, a->grp_src, a->weight);
    if (e != cudaSuccess || !in_place) return e;
    // planes: (sample, K / V, head), cut along head_dim while there are fewer of them than CTAs that fit
    int parts = 1;
    while (parts < ch_host && K.batch * 2 * K.n_kv_heads * parts < 4 * 148 && ch_host % (2 * parts) == 0) parts *= 2;
    const size_t smem = 2 * size_t(KVM_CHUNK_BYTES);
    if ((e = ensure_dynamic_smem(kv_move_kernel<T>, (int)smem)) != cudaSuccess) return e;
    return launch_kernel(kv_move_kernel<T>, dim3(K.batch * 2 * K.n_kv_heads * parts), KVM_THREADS, smem, K.stream, 1,
        static_cast<T*>(a->k_dst), static_cast<T*>(a->v_dst), da, K.n_kv_heads, K.head_dim, parts, a->vis_begin,
        a->n_text_after, K.cap_in, a->n_vis, a->n_vis_out, a->grp_off, a->grp_src, K.cap_out);
  };
  return K.dtype == LIGHTKV_BF16 ? run(__nv_bfloat16()) : run(float());
}

}  // namespace lkv
