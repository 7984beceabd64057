"""CPU oracle of the LightKV prefill-time vision-token compression step.

TEST INFRASTRUCTURE ONLY.  Plain, slow, double-precision numpy written from the
paper's method section; it shares no code with the CUDA library and must never
be imported by the product path (only tests, the smoke check and the
cpu_baseline / reference legs of the benchmark use it).

Each function names the passage of the paper it follows.  Where the paper is
silent or inconsistent the adopted reading is stated in the docstring.

Pins (see tests/test_oracle_pins.py): closed forms and special vectors for FD,
the paper's printed retention example and token counts, the printed
bipartite/full cost table, softmax identities for xi (library logsumexp,
closed form for Q = 0), convexity / weight-sum / group-mean properties of the
merge, permutation equivariance, keep = 1 identity, duplicated-token-first,
and an exhaustive brute-force matching on <= 16 tokens.
Parity unpinned by the paper (only self-consistency pins): window membership
after the first stage, multi-tile grids, output order, and the K/V operator.
A second oracle in plain C (lightkv_oracle.c), written separately, is compared
with this one in tests/test_oracle_c.py.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# Step 3 (Eq. "attention-factor"): prompt-guidance weight xi
# --------------------------------------------------------------------------

def scaled_logits(q: np.ndarray, k: np.ndarray, vis_begin: int, n_vis: int, causal: bool = True) -> np.ndarray:
    """q_i . k_j / sqrt(d_k) for the vision queries of one head, [n_vis, N]; keys a
    query may not see are set to -inf.  causal: the query at sequence index s
    sees keys 0..s (a decoder layer); otherwise it sees all N keys."""
    q = np.asarray(q, dtype=F64)
    k = np.asarray(k, dtype=F64)
    n_seq, dh = k.shape
    logits = (q[vis_begin:vis_begin + n_vis] @ k.T) / math.sqrt(dh)
    if causal:
        s = vis_begin + np.arange(n_vis)[:, None]
        logits = np.where(np.arange(n_seq)[None, :] <= s, logits, -np.inf)
    return logits


def attention_rows(q: np.ndarray, k: np.ndarray, vis_begin: int, n_vis: int, causal: bool = True) -> np.ndarray:
    """Softmax attention rows of the vision queries of one head.

    Eq. "attention-matrix": A = softmax(q K^T / sqrt(d_k)).  The equation prints
    no mask; the models it is applied to are causal decoders, so the default
    reading masks keys behind the query (causal=False is the equation as printed).
    q, k: [N, dh].  Returns A[n_vis, N] (zeros on masked keys).
    """
    logits = scaled_logits(q, k, vis_begin, n_vis, causal)
    logits = logits - logits.max(axis=1, keepdims=True)
    e = np.exp(logits)
    return e / e.sum(axis=1, keepdims=True)


def row_logsumexp(q: np.ndarray, k: np.ndarray, vis_begin: int, n_vis: int, causal: bool = True) -> np.ndarray:
    """ln sum_j exp(logit_ij) over the keys query i sees, [n_vis]: the normaliser
    of Eq. "attention-matrix" that a fused attention kernel keeps per row."""
    logits = scaled_logits(q, k, vis_begin, n_vis, causal)
    m = logits.max(axis=1)
    return m + np.log(np.exp(logits - m[:, None]).sum(axis=1))


def xi_from_attention(q: np.ndarray, k: np.ndarray, vis_begin: int, n_vis: int,
                      text_begin: int, text_end: int, causal: bool = True,
                      text_ranges: Optional[Sequence[Tuple[int, int]]] = None) -> np.ndarray:
    """xi_i = sum_h sum_{j in J} A[h, i, j]  (Eq. "attention-factor").

    q: [H, N, dh]; k: [H_kv, N, dh] (query head h reads KV head h // (H / H_kv)).
    J = [text_begin, text_end) are the prompt-token sequence indices (or the
    union of text_ranges when given); the sum runs over all H query heads with
    no averaging, as printed.
    """
    n_heads, n_kv = q.shape[0], k.shape[0]
    group = n_heads // n_kv
    ranges = [(text_begin, text_end)] if text_ranges is None else list(text_ranges)
    xi = np.zeros(n_vis, dtype=F64)
    for h in range(n_heads):
        a = attention_rows(q[h], k[h // group], vis_begin, n_vis, causal)
        for lo, hi in ranges:
            xi += a[:, lo:hi].sum(axis=1)
    return xi


# --------------------------------------------------------------------------
# Window partitioning and bipartition (Sec. "LightKV" overview; "Window
# partitioning"; Step 1)
# --------------------------------------------------------------------------

def window_of(pos: np.ndarray, tiles: Sequence[Tuple[int, int]], w: int) -> np.ndarray:
    """Window id of every token from its ORIGINAL flat grid position.

    The tokens are put back on their image grid and the grid is cut into
    w x w non-overlapping windows.  Readings: several tiles (multi-crop images,
    video frames) are windowed separately; a grid whose side is not a multiple
    of w gets balanced cells floor(row * w / rows); a token keeps its original
    position through all stages (a merged group keeps its B node's position).
    id = tile * w^2 + window_row * w + window_col.
    """
    pos = np.asarray(pos, dtype=np.int64)
    win = np.empty(pos.shape, dtype=np.int64)
    off = 0
    for t, (rows, cols) in enumerate(tiles):
        m = (pos >= off) & (pos < off + rows * cols)
        local = pos[m] - off
        r, c = local // cols, local % cols
        win[m] = t * w * w + (r * w // rows) * w + (c * w // cols)
        off += rows * cols
    return win


def bipartition(order: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Step 1: alternate assignment inside one window, tokens taken in ascending
    position.  The paper counts tokens from 1, so its "odd-indexed" tokens are
    the 1st, 3rd, ... -> set A; the 2nd, 4th, ... -> set B (A gets the extra
    node when the window holds an odd number of tokens)."""
    return order[0::2], order[1::2]


# --------------------------------------------------------------------------
# Step 2 (Eq. "similarity"): feature divergence and edge selection
# --------------------------------------------------------------------------

def feature_divergence(xa: np.ndarray, xb: np.ndarray) -> np.ndarray:
    """FD(a, b) = 1 - <x_a, x_b> / (||x_a|| ||x_b||) for all pairs, [|A|, |B|].
    A zero-norm row has cosine 0 with everything (FD = 1)."""
    xa = np.asarray(xa, dtype=F64)
    xb = np.asarray(xb, dtype=F64)
    na = np.sqrt((xa * xa).sum(axis=1))
    nb = np.sqrt((xb * xb).sum(axis=1))
    g = xa @ xb.T
    den = na[:, None] * nb[None, :]
    cos = np.divide(g, den, out=np.zeros_like(g), where=den > 0)
    return 1.0 - cos


def divergence(xa: np.ndarray, xb: np.ndarray, metric: str = "cosine") -> np.ndarray:
    """Pair scores for all (a, b), [|A|, |B|]; lower = more alike.
    "cosine": FD of Eq. "similarity" (the method).  "l2sq" / "l2": squared and plain
    Euclidean distance, the two alternatives of appendix "Influence of similarity
    metrics" (they rank pairs alike; both are kept because both are named)."""
    if metric == "cosine":
        return feature_divergence(xa, xb)
    xa = np.asarray(xa, dtype=F64)
    xb = np.asarray(xb, dtype=F64)
    diff = xa[:, None, :] - xb[None, :, :]
    sq = (diff * diff).sum(axis=2)
    if metric == "l2sq":
        return sq
    if metric == "l2":
        return np.sqrt(sq)
    raise ValueError(metric)


def removal_count(n_window: int, keep: float) -> int:
    """Tokens removed from a window of n tokens: floor(rho * n) with rho = 1 - keep,
    at most |A| = ceil(n / 2) (a step cannot remove more than half: "Limitations"),
    none when the window has no B node.

    Reading: the printed floor(rho v / 2) contradicts every count the paper
    prints (a fraction 1 - rho remains; rho = 0.5 halves 576 to 288), so the
    count is floor(rho n), evaluated as n - ceil(keep * n - 1e-9) so that the
    binary rounding of keep cannot flip the floor.
    """
    if n_window < 2:
        return 0
    r = n_window - int(math.ceil(keep * n_window - 1e-9))
    return max(0, min(r, (n_window + 1) // 2))


def select_edges(fd: np.ndarray, r: int) -> np.ndarray:
    """Adjacency M in {0,1}^{|A| x |B|} (Step 2).

    Reading: every A node keeps only its lowest-FD edge (ties -> lowest B
    index); the r A nodes whose kept edge has the lowest FD (ties -> lowest A
    index) are connected.  Several A nodes may share one B node; an A node never
    has two edges, so exactly r nodes disappear.
    """
    n_a, n_b = fd.shape
    m = np.zeros((n_a, n_b), dtype=np.int64)
    if r <= 0 or n_b == 0:
        return m
    best = np.argmin(fd, axis=1)                       # first minimum = lowest B index
    f = fd[np.arange(n_a), best]
    ranked = np.lexsort((np.arange(n_a), f))           # by f, then by A index
    for a in ranked[:r]:
        m[a, best[a]] = 1
    return m


def select_edges_literal(fd: np.ndarray, n_window: int, keep: float) -> np.ndarray:
    """Step 2 read to the letter (the alternative to select_edges): ALL |A| x |B|
    pairs are ranked by ascending FD (ties: lower A index, then lower B index) and
    the floor(rho * n / 2) lowest form T_rho, rho = 1 - keep, n = tokens of the
    window.  One-to-one matching is not enforced in either direction: an A node
    may get several edges, and the number of A nodes that disappear (those with
    at least one edge) depends on the data -- which is why the counts the paper
    prints (a fraction 1 - rho remains; 576 -> 288) cannot come from this rule.
    Kept for comparison; the library implements select_edges."""
    n_a, n_b = fd.shape
    m = np.zeros((n_a, n_b), dtype=np.int64)
    k = int(math.floor((1.0 - keep) * n_window / 2.0 + 1e-9))
    if k <= 0 or n_b == 0:
        return m
    flat = np.argsort(fd, axis=None, kind="stable")[:min(k, n_a * n_b)]   # row-major: A index, then B index
    m[np.unravel_index(flat, fd.shape)] = 1
    return m


# --------------------------------------------------------------------------
# Step 3 (Eq. "message-passing"): xi-weighted aggregation into B
# --------------------------------------------------------------------------

def message_passing(xa: np.ndarray, xb: np.ndarray, xi_a: np.ndarray, xi_b: np.ndarray,
                    m: np.ndarray) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """X_B <- (xi_B + M^T xi_A)^{-1} * (X_B . xi_B + M^T (X_A . xi_A)).

    Returns (updated X_B, weight of every A node in its group, weight of every
    B node in its group); weights are xi_i / denominator (0 for unconnected A).
    A vanishing denominator (< 1e-30) falls back to the plain group mean.
    """
    xa = np.asarray(xa, dtype=F64)
    xb = np.asarray(xb, dtype=F64)
    xi_a = np.asarray(xi_a, dtype=F64)
    xi_b = np.asarray(xi_b, dtype=F64)
    mt = m.T.astype(F64)
    den = xi_b + mt @ xi_a
    bad = den < 1e-30
    if bad.any():
        ones_a, ones_b = np.ones_like(xi_a), np.ones_like(xi_b)
        xi_a = np.where((m[:, bad].sum(axis=1) > 0), ones_a, xi_a)
        xi_b = np.where(bad, ones_b, xi_b)
        den = xi_b + mt @ xi_a
    num = xb * xi_b[:, None] + mt @ (xa * xi_a[:, None])
    xb_new = num / den[:, None]
    w_b = xi_b / den
    w_a = (m.astype(F64) @ (1.0 / den)) * xi_a
    return xb_new, w_a, w_b


# --------------------------------------------------------------------------
# One compression stage over the vision tokens of one sample (Steps 1-5)
# --------------------------------------------------------------------------

def compress_vision_literal(x: np.ndarray, pos: np.ndarray, xi: np.ndarray,
                            tiles: Sequence[Tuple[int, int]], w: int, keep: float) -> Dict[str, np.ndarray]:
    """One stage with the literal edge rule (select_edges_literal): an A node may
    send its message to several B nodes, so the map is many-to-many and is
    returned as the per-window adjacency instead of one slot per token.
    Returns x_out / pos_out (survivors in ascending position) and, per window,
    (ia, ib, M)."""
    x = np.asarray(x, dtype=F64)
    pos = np.asarray(pos, dtype=np.int64)
    xi = np.asarray(xi, dtype=F64)
    win = window_of(pos, tiles, w)
    alive = np.ones(len(x), dtype=bool)
    x_new = x.copy()
    edges = []
    for wid in np.unique(win):
        members = np.nonzero(win == wid)[0]
        members = members[np.argsort(pos[members], kind="stable")]
        ia, ib = bipartition(members)
        if len(ib) == 0:
            continue
        m = select_edges_literal(feature_divergence(x[ia], x[ib]), len(members), keep)
        xb_new, _, _ = message_passing(x[ia], x[ib], xi[ia], xi[ib], m)
        touched = m.sum(axis=0) > 0
        x_new[ib[touched]] = xb_new[touched]
        alive[ia[m.sum(axis=1) > 0]] = False
        edges.append((ia, ib, m))
    survivors = np.nonzero(alive)[0]
    survivors = survivors[np.argsort(pos[survivors], kind="stable")]
    return {"x_out": x_new[survivors], "pos_out": pos[survivors], "survivor": survivors,
            "n_out": np.int64(len(survivors)), "edges": edges}


def compress_vision(x: np.ndarray, pos: np.ndarray, xi: np.ndarray,
                    tiles: Sequence[Tuple[int, int]], w: int, keep: float,
                    metric: str = "cosine", direction: str = "a2b") -> Dict[str, np.ndarray]:
    """x [n, d], pos [n] (original flat positions, any storage order), xi [n].

    metric: pair score of Step 2 (see divergence).  direction: "a2b" passes messages
    from X_A to X_B as the method does; "b2a" is the reverse direction, which paragraph
    "Token message passing" leaves as the analogue of the forward one: the two sets swap
    roles, so B nodes are merged into their best A node and at most |B| = floor(n / 2)
    tokens of a window disappear.

    Returns
      x_out [n_out, d]  survivors (all B nodes, updated, and the unconnected A
                        nodes) in ascending original position (Step 5),
      pos_out [n_out]   their positions (a merged group keeps its B node's),
      dst [n]           output slot every input token lands in,
      weight [n]        its weight inside that slot's group (sums to 1 per slot),
      partner [n]       storage index of the B node an A token was merged into, else -1,
      survivor [n_out]  storage index of the token that owns each output slot,
      fd_best [n]       lowest FD of an A token (nan for B tokens).
    """
    x = np.asarray(x, dtype=F64)
    pos = np.asarray(pos, dtype=np.int64)
    xi = np.asarray(xi, dtype=F64)
    n = x.shape[0]
    win = window_of(pos, tiles, w)

    alive = np.ones(n, dtype=bool)
    x_new = x.copy()
    weight = np.ones(n, dtype=F64)
    partner = np.full(n, -1, dtype=np.int64)
    fd_best = np.full(n, np.nan, dtype=F64)

    for wid in np.unique(win):
        members = np.nonzero(win == wid)[0]
        members = members[np.argsort(pos[members], kind="stable")]
        ia, ib = bipartition(members)
        if len(ib) == 0:
            continue
        if direction == "b2a":
            ia, ib = ib, ia                             # sources are the B nodes, destinations the A nodes
        elif direction != "a2b":
            raise ValueError(direction)
        fd = divergence(x[ia], x[ib], metric)
        fd_best[ia] = fd.min(axis=1)
        r = min(removal_count(len(members), keep), len(ia))
        m = select_edges(fd, r)
        xb_new, w_a, w_b = message_passing(x[ia], x[ib], xi[ia], xi[ib], m)
        touched = m.sum(axis=0) > 0
        x_new[ib[touched]] = xb_new[touched]
        weight[ib] = w_b
        for a_loc, b_loc in zip(*np.nonzero(m)):
            alive[ia[a_loc]] = False                    # Step 4: delete merged A nodes
            partner[ia[a_loc]] = ib[b_loc]
            weight[ia[a_loc]] = w_a[a_loc]

    survivors = np.nonzero(alive)[0]
    survivors = survivors[np.argsort(pos[survivors], kind="stable")]
    slot = np.full(n, -1, dtype=np.int64)
    slot[survivors] = np.arange(len(survivors))
    dst = np.where(alive, slot, slot[np.where(partner >= 0, partner, 0)])
    return {"x_out": x_new[survivors], "pos_out": pos[survivors], "dst": dst,
            "weight": weight, "partner": partner, "fd_best": fd_best, "survivor": survivors,
            "n_out": np.int64(len(survivors))}


def compress_sequence(hidden: np.ndarray, vis_begin: int, n_vis: int, pos: np.ndarray,
                      xi: np.ndarray, tiles: Sequence[Tuple[int, int]], w: int, keep: float,
                      metric: str = "cosine", direction: str = "a2b") -> Dict[str, np.ndarray]:
    """Whole sequence of one sample: text rows are copied, the vision block
    [vis_begin, vis_begin + n_vis) is compressed in place of itself."""
    hidden = np.asarray(hidden, dtype=F64)
    res = compress_vision(hidden[vis_begin:vis_begin + n_vis], pos[:n_vis], xi[:n_vis], tiles, w, keep,
                          metric, direction)
    res["hidden_out"] = np.concatenate(
        [hidden[:vis_begin], res["x_out"], hidden[vis_begin + n_vis:]], axis=0)
    return res


# --------------------------------------------------------------------------
# K/V reduction (the cache shrinks together with the tokens: appendix "Method overview")
# --------------------------------------------------------------------------

def compact_kv(kv: np.ndarray, vis_begin: int, n_vis: int, dst: np.ndarray, weight: np.ndarray,
               survivor: np.ndarray, mode: str = "merge") -> np.ndarray:
    """Apply a stage's merge map to one layer's K (or V): kv [H_kv, N, dh] ->
    [H_kv, N - n_vis + n_out, dh].

    Reading (the paper gives no formula): mode "merge" uses the same
    xi-weights as the hidden states, K'_o = sum_{dst(i) = o} weight_i K_i;
    mode "gather" keeps the row of the slot's surviving token.  Text rows are
    copied.
    """
    kv = np.asarray(kv, dtype=F64)
    n_heads, n_seq, dh = kv.shape
    n_out = len(survivor)
    vis = kv[:, vis_begin:vis_begin + n_vis]
    out_vis = np.zeros((n_heads, n_out, dh), dtype=F64)
    if mode == "merge":
        for i in range(n_vis):
            out_vis[:, dst[i]] += weight[i] * vis[:, i]
    elif mode == "gather":
        out_vis[:] = vis[:, survivor]
    else:
        raise ValueError(mode)
    return np.concatenate([kv[:, :vis_begin], out_vis, kv[:, vis_begin + n_vis:]], axis=1)


# --------------------------------------------------------------------------
# Sec. "Complexity analysis" (Eq. "complexity")
# --------------------------------------------------------------------------

def vision_tokens_processed(v: float, n_layers: int, layers: Sequence[int], rho: Sequence[float]) -> float:
    """v * ( lambda_1 + sum_{i=2..s} (lambda_i - lambda_{i-1}) prod_{j<i}(1-rho_j)
            + (L - lambda_s) prod_{j<=s}(1-rho_j) )."""
    s = len(layers)
    total = float(layers[0])
    for i in range(1, s):
        total += (layers[i] - layers[i - 1]) * math.prod(1.0 - rho[j] for j in range(i))
    total += (n_layers - layers[-1]) * math.prod(1.0 - rho[j] for j in range(s))
    return v * total


def retention(n_layers: int, layers: Sequence[int], rho: Sequence[float]) -> float:
    """Fraction of the vanilla v * L vision tokens that is still processed."""
    return vision_tokens_processed(1.0, n_layers, layers, rho) / n_layers


def pair_counts(v: int, w: int = 1) -> Dict[str, float]:
    """FD evaluations: full pairwise v(v-1)/2; bipartite |A||B| per window
    (about v^2/4); windowed full pairwise v (v / w^2 - 1) / 2
    (paragraphs "Complexity" and "Window partitioning")."""
    vw = v // (w * w)
    return {"full": v * (v - 1) / 2.0,
            "bipartite": float(((vw + 1) // 2) * (vw // 2) * w * w),
            "windowed_full": 0.5 * v * (v / (w * w) - 1.0)}


# --------------------------------------------------------------------------
# Storage rounding and the whole step on a batch
# --------------------------------------------------------------------------

def to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float64 -> nearest bf16 value (ties to even), returned as float64."""
    f = np.asarray(a, dtype=np.float32)
    # double -> float first is harmless here: a value exactly between two bf16
    # neighbours after float rounding was within 2^-24 relative of that midpoint.
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(F64)


def compress_layer(hidden: np.ndarray, q: Optional[np.ndarray], k: Optional[np.ndarray],
                   pos: np.ndarray, n_vis: np.ndarray, vis_begin: int,
                   tiles: Sequence[Tuple[int, int]], w: int, keep: float,
                   text_begin: int = 0, text_end: Optional[int] = None,
                   xi: Optional[np.ndarray] = None, n_text_after: int = 0, causal: bool = True,
                   text_ranges: Optional[Sequence[Tuple[int, int]]] = None,
                   metric: str = "cosine", direction: str = "a2b") -> List[Dict[str, np.ndarray]]:
    """One compression stage on a batch (samples are independent).
    hidden [B, N, d]; q [B, H, N, dh]; k [B, H_kv, N, dh]; pos [B, cap]; n_vis [B].
    Sample b's sequence is [text (vis_begin rows) | n_vis[b] vision rows | n_text_after rows];
    rows beyond that are padding.
    xi given -> used as is; xi None -> computed from q, k (None, None -> uniform)."""
    text_end = vis_begin if text_end is None else text_end
    out = []
    for b in range(hidden.shape[0]):
        nv = int(n_vis[b])
        n_seq = vis_begin + nv + n_text_after
        if xi is not None:
            xi_b = np.asarray(xi[b][:nv], dtype=F64)
        elif q is not None:
            xi_b = xi_from_attention(q[b][:, :n_seq], k[b][:, :n_seq], vis_begin, nv, text_begin, text_end,
                                     causal, text_ranges)
        else:
            xi_b = np.ones(nv, dtype=F64)
        res = compress_sequence(hidden[b][:n_seq], vis_begin, nv, pos[b][:nv], xi_b, tiles, w, keep,
                                metric, direction)
        res["xi"] = xi_b
        out.append(res)
    return out
