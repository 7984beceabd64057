"""Seeded synthetic inputs for the LightKV compression step.

This module only *draws inputs*: smooth Gaussian random fields for the vision
rows, white noise for the text rows, rounding to bf16.  It contains none of the
method's arithmetic (no similarity, no attention, no selection, no merge) so
that both the CPU oracle and the CUDA path can be fed from it without sharing
any computation.

Recipe (stands in for LLaVA-shaped prefill activations; no dataset, no weights):
  * vision rows: per channel, white N(0,1) noise on the tile grid (padded),
    filtered with a separable Gaussian of sigma = corr_len / sqrt(2) so that the
    covariance between two patches at grid distance D is exp(-D^2 / (2 corr_len^2)),
    scaled to unit variance, plus noise_std * N(0,1);
  * video frames: F_f = c * F_{f-1} + sqrt(1 - c^2) * fresh_f (c = frame_corr);
  * text rows: N(0,1);
  * four independent tensors with that recipe: hidden [B,N,d], Q [B,H,N,dh],
    K and V [B,H_kv,N,dh]; sequence layout [text | vision];
  * everything is rounded to bf16 (round-to-nearest-even) and returned as
    float32 arrays holding exactly representable bf16 values (or left in
    float32 for the fp32 mode).
Random numbers come from numpy's counter-based Philox generator keyed by
(seed, tensor id, sample, tile), so any sub-block can be regenerated alone.
"""
from __future__ import annotations

import dataclasses
import hashlib
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

BASE_SEED = 260500789

TENSOR_HIDDEN, TENSOR_Q, TENSOR_K, TENSOR_V = 0, 1, 2, 3


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape and schedule of one synthetic workload."""
    name: str
    config_id: int
    batch: int
    tiles: Tuple[Tuple[int, int], ...]      # (rows, cols) of every image tile / frame
    n_text: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_layers: int
    layers: Tuple[int, ...]                 # Lambda: decoder layer of each stage
    windows: Tuple[int, ...]                # W: windows per axis (per tile) of each stage
    keep: Tuple[float, ...]                 # kappa_i = 1 - rho_i of each stage
    frame_corr: float = 0.0                 # correlation between consecutive tiles (video)
    corr_len: float = 3.0
    noise_std: float = 0.1

    @property
    def n_vis(self) -> int:
        return sum(r * c for r, c in self.tiles)

    @property
    def n_stages(self) -> int:
        return len(self.layers)


def _wl(**kw) -> Workload:
    return Workload(**kw)


# The five benchmark shapes (plus "4g", a stacked-tile variant of 4 whose windows
# are large enough for the similarity contraction to be compute bound) and two
# tiny ones for tests.
WORKLOADS: Dict[str, Workload] = {
    "cfg0": _wl(name="cfg0", config_id=0, batch=1, tiles=((24, 24),), n_text=32, hidden=4096,
                n_q_heads=32, n_kv_heads=32, head_dim=128, n_layers=32,
                layers=(12,), windows=(4,), keep=(0.55,)),
    "cfg1": _wl(name="cfg1", config_id=1, batch=1, tiles=((24, 24),), n_text=64, hidden=4096,
                n_q_heads=32, n_kv_heads=32, head_dim=128, n_layers=32,
                layers=(12, 18, 24), windows=(4, 2, 1), keep=(0.5, 0.5, 0.5)),
    "cfg1r": _wl(name="cfg1r", config_id=1, batch=1, tiles=((24, 24),), n_text=64, hidden=4096,
                 n_q_heads=32, n_kv_heads=32, head_dim=128, n_layers=32,
                 layers=(12, 18, 24), windows=(6, 4, 2), keep=(0.5, 0.5, 0.5)),
    "cfg2": _wl(name="cfg2", config_id=2, batch=8, tiles=((24, 24),) * 5, n_text=128, hidden=4096,
                n_q_heads=32, n_kv_heads=32, head_dim=128, n_layers=32,
                layers=(12, 18, 24), windows=(6, 4, 2), keep=(0.5, 0.5, 0.5)),
    "cfg3": _wl(name="cfg3", config_id=3, batch=32, tiles=((24, 24),), n_text=64, hidden=5120,
                n_q_heads=40, n_kv_heads=40, head_dim=128, n_layers=40,
                layers=(15, 23, 31), windows=(4, 2, 1), keep=(0.5, 0.5, 0.5)),
    "cfg4": _wl(name="cfg4", config_id=4, batch=2, tiles=((32, 32),) * 8, n_text=256, hidden=3584,
                n_q_heads=28, n_kv_heads=4, head_dim=128, n_layers=28,
                layers=(11, 16, 21), windows=(4, 2, 1), keep=(0.5, 0.5, 0.5), frame_corr=0.9),
    "cfg4g": _wl(name="cfg4g", config_id=5, batch=2, tiles=((256, 32),), n_text=256, hidden=3584,
                 n_q_heads=28, n_kv_heads=4, head_dim=128, n_layers=28,
                 layers=(11, 16, 21), windows=(4, 2, 1), keep=(0.5, 0.5, 0.5)),
    # small shapes for fast tests (several windows, ragged tails, GQA)
    "tiny": _wl(name="tiny", config_id=10, batch=2, tiles=((6, 6),), n_text=5, hidden=64,
                n_q_heads=4, n_kv_heads=2, head_dim=16, n_layers=8,
                layers=(2, 4, 6), windows=(2, 1, 1), keep=(0.5, 0.75, 0.5)),
    "small": _wl(name="small", config_id=11, batch=3, tiles=((12, 10), (9, 11)), n_text=19, hidden=264,
                 n_q_heads=6, n_kv_heads=2, head_dim=128, n_layers=12,
                 layers=(3, 6, 9), windows=(3, 2, 1), keep=(0.55, 0.6, 0.5)),
}


def workload(name: str) -> Workload:
    return WORKLOADS[name]


# --------------------------------------------------------------------------- RNG

def _generator(seed: int, *ids: int) -> np.random.Generator:
    """Counter-based generator keyed by (seed, ids...)."""
    h = hashlib.blake2b(digest_size=16)
    h.update(np.asarray([seed, *ids], dtype=np.int64).tobytes())
    key = np.frombuffer(h.digest(), dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def layer_seed(wl: Workload, layer: int, base_seed: int = BASE_SEED) -> int:
    return base_seed + 1000 * wl.config_id + layer


# ------------------------------------------------------------------- bf16 rounding

def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """float32 array -> float32 array holding the nearest bf16 values (ties to even)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    rounded = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 array of bf16-representable values -> uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bf16_from_bits(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# ------------------------------------------------------------------ random fields

def _filter_matrix(n_out: int, pad: int, sigma: float) -> np.ndarray:
    """[n_out, n_out + 2 pad] matrix applying a unit-L2-norm Gaussian kernel."""
    taps = np.arange(-pad, pad + 1, dtype=np.float64)
    g = np.exp(-taps * taps / (2.0 * sigma * sigma))
    g /= np.sqrt(np.sum(g * g))
    m = np.zeros((n_out, n_out + 2 * pad), dtype=np.float32)
    for r in range(n_out):
        m[r, r:r + 2 * pad + 1] = g
    return m


def smooth_field(rows: int, cols: int, channels: int, corr_len: float,
                 gen: np.random.Generator) -> np.ndarray:
    """Unit-variance Gaussian random field, [rows*cols, channels] float32,
    covariance exp(-D^2 / (2 corr_len^2)) between patches at grid distance D."""
    sigma = corr_len / np.sqrt(2.0)
    pad = int(np.ceil(3.0 * corr_len))
    white = gen.standard_normal((rows + 2 * pad, cols + 2 * pad, channels), dtype=np.float32)
    fr = _filter_matrix(rows, pad, sigma)
    fc = _filter_matrix(cols, pad, sigma)
    t = np.tensordot(fr, white, axes=([1], [0]))            # [rows, cols+2p, ch]
    t = np.tensordot(fc, t, axes=([1], [1]))                # [cols, rows, ch]
    return np.ascontiguousarray(t.transpose(1, 0, 2)).reshape(rows * cols, channels)


def vision_rows(wl: Workload, seed: int, tensor_id: int, sample: int, channels: int) -> np.ndarray:
    """All vision rows of one sample on the full grids: [n_vis, channels] float32
    (smooth field + white noise; frames temporally correlated when frame_corr > 0)."""
    out = np.empty((wl.n_vis, channels), dtype=np.float32)
    off = 0
    prev = None
    c = float(wl.frame_corr)
    for t, (rows, cols) in enumerate(wl.tiles):
        gen = _generator(seed, tensor_id, sample, t)
        f = smooth_field(rows, cols, channels, wl.corr_len, gen)
        if c > 0.0 and prev is not None and prev.shape == f.shape:
            f = np.float32(c) * prev + np.float32(np.sqrt(1.0 - c * c)) * f
        prev = f
        noise = gen.standard_normal(f.shape, dtype=np.float32)
        out[off:off + rows * cols] = f + np.float32(wl.noise_std) * noise
        off += rows * cols
    return out


def text_rows(wl: Workload, seed: int, tensor_id: int, sample: int, channels: int) -> np.ndarray:
    gen = _generator(seed, tensor_id, sample, 1_000_003)
    return gen.standard_normal((wl.n_text, channels), dtype=np.float32)


def make_layer_inputs(wl: Workload, stage: int, pos: Optional[Sequence[np.ndarray]] = None,
                      dtype: str = "bf16", tensors: Sequence[str] = ("hidden", "q", "k", "v"),
                      base_seed: int = BASE_SEED, samples: Optional[Sequence[int]] = None
                      ) -> Dict[str, object]:
    """Inputs of compression stage `stage` (decoder layer wl.layers[stage]).

    pos: per sample, ascending int array of the original flat grid positions of
    the vision tokens still alive (None = all of them, i.e. the first stage).
    A fresh field is drawn with that layer's seed on the full grids and sampled
    at those positions.  Returns float32 arrays (bf16-representable when
    dtype == "bf16"), zero padded to the longest sample:
      hidden [B, N, d];  q [B, H, N, dh];  k, v [B, H_kv, N, dh];  N = n_text + max n_vis
      pos [B, cap] int32 (padded with -1);  n_vis [B] int32.
    """
    samples = list(range(wl.batch)) if samples is None else list(samples)
    nb = len(samples)
    if pos is None:
        pos = [np.arange(wl.n_vis, dtype=np.int32) for _ in samples]
    pos = [np.asarray(p, dtype=np.int32) for p in pos]
    n_vis = np.asarray([len(p) for p in pos], dtype=np.int32)
    cap = int(n_vis.max()) if nb else 0
    n_seq = wl.n_text + cap
    seed = layer_seed(wl, wl.layers[stage], base_seed)
    rnd = round_to_bf16 if dtype == "bf16" else (lambda a: np.ascontiguousarray(a, dtype=np.float32))

    out: Dict[str, object] = {"n_vis": n_vis, "n_text": wl.n_text, "vis_begin": wl.n_text}
    pos_pad = np.full((nb, cap), -1, dtype=np.int32)
    for i, p in enumerate(pos):
        pos_pad[i, :len(p)] = p
    out["pos"] = pos_pad

    spec = {"hidden": (TENSOR_HIDDEN, 1, wl.hidden), "q": (TENSOR_Q, wl.n_q_heads, wl.head_dim),
            "k": (TENSOR_K, wl.n_kv_heads, wl.head_dim), "v": (TENSOR_V, wl.n_kv_heads, wl.head_dim)}
    for name in tensors:
        tid, heads, width = spec[name]
        ch = heads * width
        if name == "hidden":
            arr = np.zeros((nb, n_seq, ch), dtype=np.float32)
        else:
            arr = np.zeros((nb, heads, n_seq, width), dtype=np.float32)
        for i, b in enumerate(samples):
            txt = rnd(text_rows(wl, seed, tid, b, ch))
            vis = rnd(vision_rows(wl, seed, tid, b, ch)[pos[i]])
            nv = len(pos[i])
            if name == "hidden":
                arr[i, :wl.n_text] = txt
                arr[i, wl.n_text:wl.n_text + nv] = vis
            else:
                arr[i, :, :wl.n_text] = txt.reshape(wl.n_text, heads, width).transpose(1, 0, 2)
                arr[i, :, wl.n_text:wl.n_text + nv] = vis.reshape(nv, heads, width).transpose(1, 0, 2)
        out[name] = arr
    return out
