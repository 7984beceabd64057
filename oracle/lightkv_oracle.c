/*
 * Plain C restatement of the LightKV compression step, one sample at a time, double precision, simple loops.
 *
 * TEST INFRASTRUCTURE ONLY: a second, separately written oracle.  It follows the same passages of the paper as
 * oracle/lightkv_oracle.py (Eq. "attention-matrix" / "attention-factor" for xi, "Window partitioning" and Step 1
 * for windows and the bipartition, Eq. "similarity" and Step 2 for the feature divergence and the choice of edges,
 * Eq. "message-passing" and Steps 3-5 for the merge) and shares no code with it or with the CUDA library.  The
 * tests compare the two oracles with each other; bench.py may time this one as the single-threaded CPU baseline.
 * Readings of the paper are the ones listed in the Python oracle's docstrings (one edge per A node, floor(rho n)
 * removals per window capped at |A|, 1-based "odd-indexed" tokens form A, ascending-position output order, ...).
 *
 * Build: gcc -O2 -shared -fPIC -o liboracle_c.so lightkv_oracle.c -lm
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

/* xi_i = sum_h sum_{j in J} softmax_j(q_i . k_j / sqrt(dh)) over the keys query i sees.
 * q [H][N][dh], k [H_kv][N][dh] (row-major doubles); vision queries are rows vis_begin .. vis_begin + n_vis - 1;
 * J is the union of n_ranges index ranges [lo, hi); causal != 0: query at index s sees keys 0..s. */
void oracle_c_xi(const double* q, const double* k, int n_heads, int n_kv, int n_seq, int dh, int vis_begin, int n_vis,
                 const int* ranges, int n_ranges, int causal, double* xi) {
  const int group = n_heads / n_kv;
  const double scale = 1.0 / sqrt((double)dh);
  double* logit = (double*)malloc(sizeof(double) * (size_t)n_seq);
  for (int i = 0; i < n_vis; ++i) xi[i] = 0.0;
  for (int h = 0; h < n_heads; ++h) {
    const double* kh = k + (size_t)(h / group) * n_seq * dh;
    for (int i = 0; i < n_vis; ++i) {
      const int s = vis_begin + i;
      const int last = causal ? s : n_seq - 1;
      const double* qi = q + ((size_t)h * n_seq + s) * dh;
      double mx = -INFINITY;
      for (int j = 0; j <= last; ++j) {
        double acc = 0.0;
        for (int c = 0; c < dh; ++c) acc += qi[c] * kh[(size_t)j * dh + c];
        logit[j] = acc * scale;
        if (logit[j] > mx) mx = logit[j];
      }
      double den = 0.0, num = 0.0;
      for (int j = 0; j <= last; ++j) {
        const double p = exp(logit[j] - mx);
        den += p;
        for (int r = 0; r < n_ranges; ++r)
          if (j >= ranges[2 * r] && j < ranges[2 * r + 1]) { num += p; break; }
      }
      xi[i] += num / den;
    }
  }
  free(logit);
}

static int window_id(int pos, const int* tiles, int n_tiles, int w) {
  int off = 0;
  for (int t = 0; t < n_tiles; ++t) {
    const int rows = tiles[2 * t], cols = tiles[2 * t + 1];
    if (pos >= off && pos < off + rows * cols) {
      const int local = pos - off, r = local / cols, c = local % cols;
      return t * w * w + (r * w / rows) * w + (c * w / cols);
    }
    off += rows * cols;
  }
  return -1;
}

static int removal_count(int n, double keep) {
  if (n < 2) return 0;
  int r = n - (int)ceil(keep * n - 1e-9);
  const int na = (n + 1) / 2;
  if (r < 0) r = 0;
  if (r > na) r = na;
  return r;
}

/* One compression stage on the vision tokens of one sample (Steps 1-5, direction A -> B, cosine FD).
 * x [n][d], pos [n] strictly ascending, xi [n].  Outputs: x_out [n][d] (first *n_out rows used), pos_out [n],
 * dst [n] (output slot of every token), weight [n] (its weight inside the slot's group).  Returns 0. */
int oracle_c_compress(const double* x, const int* pos, const double* xi, int n, int d, const int* tiles, int n_tiles,
                      int w, double keep, double* x_out, int* pos_out, int* dst, double* weight, int* n_out) {
  const int n_win = n_tiles * w * w;
  int* win = (int*)malloc(sizeof(int) * (size_t)n);
  int* partner = (int*)malloc(sizeof(int) * (size_t)n);
  int* members = (int*)malloc(sizeof(int) * (size_t)n);
  double* best_fd = (double*)malloc(sizeof(double) * (size_t)n);
  int* best_b = (int*)malloc(sizeof(int) * (size_t)n);
  double* norm = (double*)malloc(sizeof(double) * (size_t)n);
  for (int i = 0; i < n; ++i) {
    win[i] = window_id(pos[i], tiles, n_tiles, w);
    partner[i] = -1;
    double ss = 0.0;
    for (int c = 0; c < d; ++c) ss += x[(size_t)i * d + c] * x[(size_t)i * d + c];
    norm[i] = sqrt(ss);
  }
  for (int wid = 0; wid < n_win; ++wid) {
    int m = 0;
    for (int i = 0; i < n; ++i) if (win[i] == wid) members[m++] = i;      /* ascending position = storage order */
    const int na = (m + 1) / 2, nb = m / 2;
    if (nb == 0) continue;
    /* A = members 0, 2, 4, ...; B = members 1, 3, 5, ...; lowest-FD B node of every A node (first minimum) */
    for (int ia = 0; ia < na; ++ia) {
      const int a = members[2 * ia];
      double best = INFINITY; int arg = -1;
      for (int ib = 0; ib < nb; ++ib) {
        const int b = members[2 * ib + 1];
        double g = 0.0;
        for (int c = 0; c < d; ++c) g += x[(size_t)a * d + c] * x[(size_t)b * d + c];
        const double den = norm[a] * norm[b];
        const double fd = 1.0 - (den > 0.0 ? g / den : 0.0);
        if (fd < best) { best = fd; arg = b; }
      }
      best_fd[a] = best; best_b[a] = arg;
    }
    /* the r A nodes with the lowest (FD, index) are connected */
    const int r = removal_count(m, keep);
    for (int pick = 0; pick < r; ++pick) {
      int arg = -1;
      for (int ia = 0; ia < na; ++ia) {
        const int a = members[2 * ia];
        if (partner[a] >= 0) continue;
        if (arg < 0 || best_fd[a] < best_fd[arg]) arg = a;      /* ties keep the earlier A node */
      }
      partner[arg] = best_b[arg];
    }
  }
  /* survivors in ascending position, merged rows */
  int o = 0;
  int* slot = (int*)malloc(sizeof(int) * (size_t)n);
  for (int i = 0; i < n; ++i) if (partner[i] < 0) { slot[i] = o; pos_out[o] = pos[i]; ++o; }
  *n_out = o;
  for (int i = 0; i < n; ++i) dst[i] = partner[i] < 0 ? slot[i] : slot[partner[i]];
  for (int s = 0; s < o; ++s) for (int c = 0; c < d; ++c) x_out[(size_t)s * d + c] = 0.0;
  double* den = (double*)calloc((size_t)o, sizeof(double));
  int* size = (int*)calloc((size_t)o, sizeof(int));
  for (int i = 0; i < n; ++i) { den[dst[i]] += xi[i]; size[dst[i]] += 1; }
  for (int i = 0; i < n; ++i) {
    const int s = dst[i];
    weight[i] = den[s] < 1e-30 ? 1.0 / size[s] : xi[i] / den[s];       /* vanishing sum: plain group mean */
  }
  for (int i = 0; i < n; ++i) {
    const int s = dst[i];
    if (size[s] == 1) { memcpy(x_out + (size_t)s * d, x + (size_t)i * d, sizeof(double) * (size_t)d); continue; }
    for (int c = 0; c < d; ++c) x_out[(size_t)s * d + c] += weight[i] * x[(size_t)i * d + c];
  }
  free(win); free(partner); free(members); free(best_fd); free(best_b); free(norm); free(slot); free(den); free(size);
  return 0;
}

/* K'_o = sum_{dst(i) = o} weight_i K_i per head (the same map as the hidden states); kv [H][n][dh] -> out [H][n_out][dh]. */
void oracle_c_compact(const double* kv, int n_heads, int n, int dh, const int* dst, const double* weight, int n_out, double* out) {
  for (size_t i = 0; i < (size_t)n_heads * n_out * dh; ++i) out[i] = 0.0;
  for (int h = 0; h < n_heads; ++h)
    for (int i = 0; i < n; ++i)
      for (int c = 0; c < dh; ++c)
        out[((size_t)h * n_out + dst[i]) * dh + c] += weight[i] * kv[((size_t)h * n + i) * dh + c];
}
