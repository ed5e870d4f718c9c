"""Seeded synthetic video-shaped inputs and the five workload descriptors.

This module is the only code shared by the CUDA path's tests/bench and the CPU
oracle's tests.  It holds no arithmetic of the method (no attention, score,
selection or mask logic): it only draws Q/K/V tensors and describes sequences.

Sequences follow the token layout the method's mask presumes (Sec. 3.2: "first
frame", "current frame", "corresponding token in the previous frame"):
    [n_prefix text tokens][F frames x (grid_h x grid_w) visual tokens][n_suffix text tokens]
with visual tokens in raster order inside a frame.

Values: every element is N(0,1) from a counter-based generator (splitmix64 of
(seed, tensor id, layer) plus the element's pair index, then Box-Muller in
float64), so an element does not depend on how much else is generated.  On top
of that sits the salient-direction structure of the workload descriptions: 5 %
of visual positions (a hash of seed, request, position; the same in every layer
and head) get K += 3 u, and the last 16 queries of each request get Q += u,
with one unit vector u per (layer, KV head).  Values are rounded float64 ->
float32 -> (for bf16 workloads) bfloat16 round-to-nearest-even.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor
from typing import List, Optional, Sequence, Tuple

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLD = np.uint64(0x9E3779B97F4A7C15)
_C1 = np.uint64(0xBF58476D1CE4E5B9)
_C2 = np.uint64(0x94D049BB133111EB)

TENSOR_Q, TENSOR_K, TENSOR_V, TENSOR_U, TENSOR_SALIENT, TENSOR_SHAPE = 1, 2, 3, 4, 5, 6


def splitmix64(x: np.ndarray) -> np.ndarray:
    """The splitmix64 finaliser on uint64 arrays (wrap-around arithmetic)."""
    with np.errstate(over="ignore"):
        z = (x + _GOLD).astype(np.uint64)
        z = (z ^ (z >> np.uint64(30))) * _C1
        z = (z ^ (z >> np.uint64(27))) * _C2
        return z ^ (z >> np.uint64(31))


def _stream_key(seed: int, tensor_id: int, layer: int) -> np.uint64:
    a = splitmix64(np.array([seed], dtype=np.uint64))
    with np.errstate(over="ignore"):
        b = splitmix64(a ^ (np.uint64(tensor_id) * _C2))
        c = splitmix64(b + np.uint64(layer))
    return c[0]


def normal_pairs(key: np.uint64, first_pair: int, n_pairs: int) -> np.ndarray:
    """2*n_pairs N(0,1) float64 values: pair p yields (r cos, r sin) at 2p, 2p+1."""
    with np.errstate(over="ignore"):
        ctr = np.arange(first_pair, first_pair + n_pairs, dtype=np.uint64)
        h1 = splitmix64(key + ctr)
        h2 = splitmix64(h1)
    u1 = ((h1 >> np.uint64(11)).astype(np.float64) + 1.0) * (1.0 / 9007199254740992.0)
    u2 = (h2 >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)
    r = np.sqrt(-2.0 * np.log(u1))
    th = (2.0 * np.pi) * u2
    out = np.empty(2 * n_pairs, dtype=np.float64)
    out[0::2] = r * np.cos(th)
    out[1::2] = r * np.sin(th)
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest even."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rnd = ((b >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((b + rnd) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclasses.dataclass(frozen=True)
class STMask:
    """Parameters of the spatial-temporal mask; the defaults are the paper's mask
    (Sec. 3.2): first frame + whole current frame + same cell of the previous frame."""
    grid_h: int
    grid_w: int
    anchor_frames: int = 1
    spatial_radius: int = -1
    temporal_depth: int = 1
    temporal_stride: int = 1
    temporal_radius: int = 0
    tile: int = 128
    dense_causal: bool = False
    local_window: int = 0        # > 0: also the most recent positions (Local Attention of App. A.3)
    atrous_dilation: int = 0     # > 0: also every n-th earlier position (Atrous Attention of App. A.3)
    coarse: bool = False         # widen the mask to whole tile x tile blocks (block-sparse reading)


def mask_variant(name: str, grid_h: int, grid_w: int, tile: int = 128, coarse: bool = False, local_window: int = 64,
                 atrous_dilation: int = 4) -> STMask:
    """The sparse-attention variants the paper compares (App. A.3, Table 7), as parameter settings:
    "st" the paper's mask; "spatial" its spatial path alone (first frame + current frame); "temporal" its temporal
    path alone (first frame + the same cell of the previous frame, and the token itself); "local" the most recent
    `local_window` positions; "atrous" every `atrous_dilation`-th earlier position.  Prefix tokens stay visible and
    text rows dense in all of them."""
    kw = dict(tile=tile, coarse=coarse)
    if name == "st":
        return STMask(grid_h, grid_w, **kw)
    if name == "spatial":
        return STMask(grid_h, grid_w, 1, -1, 0, 1, 0, **kw)
    if name == "temporal":
        return STMask(grid_h, grid_w, 1, 0, 1, 1, 0, **kw)
    if name == "local":
        return STMask(grid_h, grid_w, 0, 0, 0, 1, 0, local_window=local_window, **kw)
    if name == "atrous":
        return STMask(grid_h, grid_w, 0, 0, 0, 1, 0, atrous_dilation=atrous_dilation, **kw)
    raise ValueError(f"no mask variant {name!r}")


@dataclasses.dataclass(frozen=True)
class Batch:
    """Packed variable-length batch of video+text sequences."""
    seq_lens: Tuple[int, ...]
    n_prefix: Tuple[int, ...]
    n_frames: Tuple[int, ...]
    grid_h: int
    grid_w: int

    @property
    def n_req(self) -> int:
        return len(self.seq_lens)

    @property
    def total_tokens(self) -> int:
        return int(sum(self.seq_lens))

    @property
    def cu_seqlens(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.seq_lens)]).astype(np.int32)

    def n_suffix(self, r: int) -> int:
        return self.seq_lens[r] - self.n_prefix[r] - self.n_frames[r] * self.grid_h * self.grid_w


def make_batch(n_prefix: Sequence[int], n_frames: Sequence[int], n_suffix: Sequence[int],
               grid_h: int, grid_w: int) -> Batch:
    n = grid_h * grid_w
    lens = tuple(int(p + f * n + s) for p, f, s in zip(n_prefix, n_frames, n_suffix))
    return Batch(lens, tuple(int(p) for p in n_prefix), tuple(int(f) for f in n_frames), grid_h, grid_w)


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    dtype: str                   # "bf16" | "fp32"
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_layers: int                # layers that run attention
    scored_layers: Tuple[int, ...]
    compacted_layers: Tuple[int, ...]
    batch: Batch
    mask: STMask
    window: int
    keep_ratio: float


def _ragged_draw(seed: int, n_req: int) -> Tuple[List[int], List[int]]:
    key = _stream_key(seed, TENSOR_SHAPE, 0)
    with np.errstate(over="ignore"):
        h = splitmix64(key + np.arange(2 * n_req, dtype=np.uint64))
    frames = [int(8 + (int(h[2 * r]) % 57)) for r in range(n_req)]          # uniform 8..64
    text = [int(32 + (int(h[2 * r + 1]) % 225)) for r in range(n_req)]      # uniform 32..256
    return frames, text


def workload(cfg: int, **over) -> Workload:
    """The five workloads (0 tiny fp32, 1 VideoLLaMA2-shaped, 2 Qwen2.5-VL-shaped,
    3 long video, 4 ragged serving batch).  `over` replaces Workload fields."""
    seed = 20251025 + cfg
    if cfg == 0:
        w = Workload("cfg0_tiny_fp32", seed, "fp32", 2, 1, 64, 1, (0,), (0,),
                     make_batch([16], [4], [16], 8, 8), STMask(8, 8, tile=16), 16, 0.2)
    elif cfg == 1:
        w = Workload("cfg1_videollama2", seed, "bf16", 32, 8, 128, 32, (0,), tuple(range(1, 32)),
                     make_batch([64], [16], [64], 12, 12), STMask(12, 12, tile=64), 64, 0.2)
    elif cfg == 2:
        w = Workload("cfg2_qwen25vl", seed, "bf16", 28, 4, 128, 28, (0, 1), tuple(range(2, 28)),
                     make_batch([64], [32], [64], 16, 16), STMask(16, 16, tile=128), 64, 0.2)
    elif cfg == 3:
        w = Workload("cfg3_long_video", seed, "bf16", 28, 4, 128, 1, (0,), (0,),
                     make_batch([0], [64], [256], 24, 24), STMask(24, 24, tile=128), 256, 0.2)
    elif cfg == 4:
        frames, text = _ragged_draw(seed, 8)
        w = Workload("cfg4_ragged_batch", seed, "bf16", 28, 4, 128, 1, (0,), tuple(range(27)),
                     make_batch([0] * 8, frames, text, 16, 16), STMask(16, 16, tile=128), 32, 0.2)
    else:
        raise ValueError(f"no workload {cfg}")
    return dataclasses.replace(w, **over) if over else w


def salient_positions(seed: int, batch: Batch, prob: float = 0.05) -> np.ndarray:
    """Boolean [T]: visual positions marked salient (same in every layer and head)."""
    out = np.zeros(batch.total_tokens, dtype=bool)
    cu = batch.cu_seqlens
    n = batch.grid_h * batch.grid_w
    thresh = int(prob * 2.0 ** 53)
    for r in range(batch.n_req):
        key = _stream_key(seed, TENSOR_SALIENT, r)
        nv = batch.n_frames[r] * n
        with np.errstate(over="ignore"):
            h = splitmix64(key + np.arange(nv, dtype=np.uint64))
        lo = int(cu[r]) + batch.n_prefix[r]
        out[lo:lo + nv] = (h >> np.uint64(11)).astype(np.int64) < thresh
    return out


def salient_directions(seed: int, layer: int, n_kv_heads: int, head_dim: int) -> np.ndarray:
    """[n_kv_heads, head_dim] float64 unit vectors u[layer, g]."""
    key = _stream_key(seed, TENSOR_U, layer)
    z = normal_pairs(key, 0, n_kv_heads * head_dim // 2).reshape(n_kv_heads, head_dim)
    return z / np.sqrt((z * z).sum(axis=1, keepdims=True))


_CHUNK_TOKENS = 1 << 8


def _draw(key: np.uint64, t0: int, t1: int, n_heads: int, d: int) -> np.ndarray:
    per_tok = n_heads * d // 2
    return normal_pairs(key, t0 * per_tok, (t1 - t0) * per_tok).reshape(t1 - t0, n_heads, d)


def make_qkv(wl: Workload, layer: int, which: str = "qkv", k_boost: float = 3.0, q_boost: float = 1.0,
             pool: Optional[ThreadPoolExecutor] = None):
    """Draw layer `layer`'s tensors.  Returns a dict with float32 arrays 'q' [T,H,d],
    'k','v' [T,H_kv,d]; for bf16 workloads the values are already rounded to bf16
    (exactly representable), and 'q_bits' etc. hold the uint16 bit patterns."""
    b = wl.batch
    t_tot, h, hkv, d = b.total_tokens, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
    g = h // hkv
    u = salient_directions(wl.seed, layer, hkv, d)
    sal = salient_positions(wl.seed, b)
    cu = b.cu_seqlens
    last_q = np.zeros(t_tot, dtype=bool)
    for r in range(b.n_req):
        last_q[max(int(cu[r]), int(cu[r + 1]) - 16):int(cu[r + 1])] = True
    out = {}
    spec = {"q": (TENSOR_Q, h), "k": (TENSOR_K, hkv), "v": (TENSOR_V, hkv)}
    for name in ("q", "k", "v"):
        if name not in which:
            continue
        tid, nh = spec[name]
        key = _stream_key(wl.seed, tid, layer)
        arr = np.empty((t_tot, nh, d), dtype=np.float32)

        def job(t0, name=name, nh=nh, key=key, arr=arr):
            t1 = min(t_tot, t0 + _CHUNK_TOKENS)
            x = _draw(key, t0, t1, nh, d)
            if name == "k":
                x[sal[t0:t1]] += k_boost * u[None, :, :]
            elif name == "q":
                x[last_q[t0:t1]] += q_boost * np.repeat(u, g, axis=0)[None, :, :]
            arr[t0:t1] = x.astype(np.float32)

        starts = range(0, t_tot, _CHUNK_TOKENS)
        if pool is not None:
            list(pool.map(job, starts))
        else:
            for s in starts:
                job(s)
        if wl.dtype == "bf16":
            bits = f32_to_bf16_bits(arr)
            out[name + "_bits"] = bits
            arr = bf16_bits_to_f32(bits)
        out[name] = arr
    return out
