"""Seeded synthetic prompts shaped like LOOK-M's multimodal long-context workloads.

This module only *draws inputs*: interleaved text/image prompt layouts, a modality mask, and
bf16-exact Q/K/V tensors.  It contains none of the compression method's arithmetic and depends on
numpy alone, so the CUDA path and the CPU oracle can both be fed from it without sharing code.

Randomness comes from one counter-based generator (a splitmix64-style mixer over
``hash(stream key) + counter``) followed by Box-Muller, so a value depends only on its stream key
and position, never on a library's RNG version.  Every tensor is rounded to bf16
(round-to-nearest-even) on the host; the returned ``uint16`` arrays hold those bf16 bit patterns
and :func:`bf16_to_f32` widens them exactly.

The workloads stand in for MileBench prompts run through LLaVA-1.5-shaped models (the paper's
evaluation setting, Section 4): many 576-token images interleaved with short text segments.
Image keys are drawn around 24 cluster centres per (image, KV head) so that neighbouring patches
are redundant, which is the structure the method's eviction and merging exploit.
"""
from __future__ import annotations

import os
from dataclasses import dataclass, field
from typing import List, Sequence, Tuple

import numpy as np

IMAGE_TOKENS = 576          # tokens per image (24 x 24 patches)
CLUSTERS_PER_IMAGE = 24     # one centre per patch row
MERGE_AVERAGE, MERGE_PIVOTAL, MERGE_WEIGHTED = 0, 1, 2

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

# tensor ids used in stream keys
_T_Q, _T_K, _T_V, _T_CENTRE, _T_SEGMENTS, _T_OUTLIER, _T_LENGTH = 1, 2, 3, 4, 5, 6, 7


def _mix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser, vectorised over uint64 (wrap-around arithmetic intended)."""
    x = x.copy()
    x ^= x >> np.uint64(30)
    x *= _M1
    x ^= x >> np.uint64(27)
    x *= _M2
    x ^= x >> np.uint64(31)
    return x


def stream_key(*parts: int) -> np.uint64:
    """Fold a tuple of small integers into one 64-bit stream key."""
    with np.errstate(over="ignore"):
        h = np.array([0x243F6A8885A308D3], dtype=np.uint64)
        for p in parts:
            h = _mix64(h + np.uint64(int(p) & 0xFFFFFFFFFFFFFFFF) * _GOLDEN + np.uint64(1))
        return h[0]


def uniform_u64(key: np.uint64, n: int, offset: int = 0) -> np.ndarray:
    """n raw 64-bit draws of stream `key`, counters offset .. offset+n-1."""
    with np.errstate(over="ignore"):
        c = np.arange(offset, offset + n, dtype=np.uint64)
        return _mix64(_mix64(np.uint64(key) + c * _GOLDEN))


def uniform_int(key: np.uint64, n: int, lo: int, hi: int, offset: int = 0) -> np.ndarray:
    """n integers uniform on [lo, hi] (inclusive)."""
    span = np.uint64(hi - lo + 1)
    return (uniform_u64(key, n, offset) >> np.uint64(11)) % span + np.uint64(lo)


def _normal_chunk(key: np.uint64, s: int, m: int, out: np.ndarray) -> None:
    x = uniform_u64(key, m, s)
    u1 = ((x >> np.uint64(32)).astype(np.float64) + 0.5) * (1.0 / 4294967296.0)
    u2 = ((x & np.uint64(0xFFFFFFFF)).astype(np.float64) + 0.5) * (1.0 / 4294967296.0)
    r = np.sqrt(-2.0 * np.log(u1))
    t = (2.0 * np.pi) * u2
    out[2 * s:2 * (s + m):2] = r * np.cos(t)
    out[2 * s + 1:2 * (s + m):2] = r * np.sin(t)


def normal(key: np.uint64, n: int) -> np.ndarray:
    """n standard normal draws (float64) from stream `key` by Box-Muller.

    Counter c yields draws 2c and 2c+1, so the result does not depend on how the work is chunked;
    large requests are spread over a thread pool (numpy releases the GIL inside each chunk).
    """
    half = (n + 1) // 2
    out = np.empty(2 * half, dtype=np.float64)
    chunk = 1 << 20
    starts = list(range(0, half, chunk))
    if len(starts) <= 2:
        for s in starts:
            _normal_chunk(key, s, min(chunk, half - s), out)
    else:
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(max_workers=_workers()) as ex:
            list(ex.map(lambda s: _normal_chunk(key, s, min(chunk, half - s), out), starts))
    return out[:n]


def _workers() -> int:
    try:
        return max(1, min(32, len(os.sched_getaffinity(0))))
    except AttributeError:
        return max(1, min(32, os.cpu_count() or 1))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns the uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    flat = x.reshape(-1).view(np.uint32)
    out = np.empty(flat.shape[0], dtype=np.uint16)

    def piece(s):
        b = flat[s:s + (1 << 22)]
        out[s:s + (1 << 22)] = ((b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1)))
                                >> np.uint32(16)).astype(np.uint16)

    starts = list(range(0, flat.shape[0], 1 << 22))
    if len(starts) <= 1:
        for s0 in starts:
            piece(s0)
    else:
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(max_workers=_workers()) as ex:
            list(ex.map(piece, starts))
    return out.reshape(x.shape)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to float32 exactly."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ---------------------------------------------------------------------------------------------
# prompt layouts
# ---------------------------------------------------------------------------------------------

def text_segments(key: np.uint64, n_segments: int, total: int, lo: int, hi: int) -> List[int]:
    """Segment lengths uniform on [lo, hi], repaired +-1 round-robin until they sum to `total`."""
    if not (n_segments * lo <= total <= n_segments * hi):
        raise ValueError("text total not reachable within the segment bounds")
    seg = [int(v) for v in uniform_int(key, n_segments, lo, hi)]
    i = 0
    while sum(seg) != total:
        step = 1 if sum(seg) < total else -1
        if lo <= seg[i] + step <= hi:
            seg[i] += step
        i = (i + 1) % n_segments
    return seg


def interleave(n_images: int, segments: Sequence[int]) -> np.ndarray:
    """Modality mask (uint8, 1 = image token) of the prompt T I T I ... T."""
    assert len(segments) == n_images + 1
    parts = []
    for s in range(n_images):
        parts.append(np.zeros(segments[s], dtype=np.uint8))
        parts.append(np.ones(IMAGE_TOKENS, dtype=np.uint8))
    parts.append(np.zeros(segments[-1], dtype=np.uint8))
    return np.concatenate(parts)


@dataclass
class Request:
    seq_len: int
    n_images: int
    segments: List[int]
    budget: int
    window: int
    merge_mode: int
    mask: np.ndarray = field(repr=False, default=None)


@dataclass
class Workload:
    name: str
    config_id: int
    seed: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    k_outliers: bool
    requests: List[Request]

    @property
    def total_tokens(self) -> int:
        return sum(r.seq_len for r in self.requests)

    @property
    def cu_seqlens(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum([r.seq_len for r in self.requests])]).astype(np.int32)


def _request(key_parts: Tuple[int, ...], seq_len: int, n_images: int, seg_lo: int, seg_hi: int,
             ratio: float, window: int, merge_mode: int, fixed_segments=None) -> Request:
    text_total = seq_len - n_images * IMAGE_TOKENS
    if fixed_segments is not None:
        seg = list(fixed_segments)
    else:
        seg = text_segments(stream_key(*key_parts, _T_SEGMENTS), n_images + 1, text_total, seg_lo, seg_hi)
    assert sum(seg) == text_total
    return Request(seq_len=seq_len, n_images=n_images, segments=seg, budget=int(ratio * seq_len),
                   window=window, merge_mode=merge_mode, mask=interleave(n_images, seg))


def config1(seed: int = 0) -> Workload:
    """2048-token prompt: 3 images and 4 text segments of 80 tokens; 8 heads; averaged merging."""
    r = _request((seed, 1, 0), 2048, 3, 80, 80, 0.2, 32, MERGE_AVERAGE, fixed_segments=[80] * 4)
    return Workload("c1_2k_8h", 1, seed, 1, 8, 8, 128, False, [r])


def config2(seed: int = 0, merge_mode: int = MERGE_AVERAGE, ratio: float = 0.2) -> Workload:
    """LLaVA-1.5-7B shape: 32 layers x 32 heads, 8192-token prompt of 12 images + 1280 text tokens."""
    r = _request((seed, 2, 0), 8192, 12, 40, 200, ratio, 32, merge_mode)
    return Workload("c2_8k_7b", 2, seed, 32, 32, 32, 128, True, [r])


def config3(seed: int = 0, ratio: float = 0.2) -> Workload:
    """LLaVA-1.5-13B shape: 40 layers x 40 heads, 16384-token prompt of 24 images + 2560 text tokens."""
    r = _request((seed, 3, 0), 16384, 24, 40, 200, ratio, 64, MERGE_WEIGHTED)
    return Workload("c3_16k_13b", 3, seed, 40, 40, 40, 128, False, [r])


def config4(seed: int = 0) -> Workload:
    """Grouped-query shape: 32 query heads on 8 KV heads, 32768-token prompt of 52 images."""
    r = _request((seed, 4, 0), 32768, 52, 20, 120, 0.2, 64, MERGE_PIVOTAL)
    return Workload("c4_32k_gqa", 4, seed, 32, 32, 8, 128, False, [r])


def config5(seed: int = 0, n_requests: int = 16) -> Workload:
    """Ragged serving batch on the 7B shape: prompt lengths uniform on [2048, 16384]."""
    reqs: List[Request] = []
    draw = 0
    lkey = stream_key(seed, 5, _T_LENGTH)
    while len(reqs) < n_requests:
        L = int(uniform_int(lkey, 1, 2048, 16384, offset=draw)[0])
        draw += 1
        ok = [n for n in range(2, 25)
              if L - n * IMAGE_TOKENS > 0 and 0.10 <= (L - n * IMAGE_TOKENS) / L <= 0.20]
        if not ok:
            continue
        n_img = max(ok)
        text_total = L - n_img * IMAGE_TOKENS
        mean = text_total / (n_img + 1)
        lo, hi = int(np.floor(0.5 * mean)), int(np.ceil(1.5 * mean))
        r = len(reqs)
        reqs.append(_request((seed, 5, r), L, n_img, lo, hi, 0.2, 32, r % 3))
    return Workload("c5_ragged_7b", 5, seed, 32, 32, 32, 128, False, reqs)


def tiny(seq_len: int, n_q_heads: int, n_kv_heads: int, budget: int, window: int, merge_mode: int,
         image_spans: Sequence[Tuple[int, int]] = (), seed: int = 0, head_dim: int = 128) -> Workload:
    """Small ad-hoc workload for tests: i.i.d. tokens with the given [start, end) image spans."""
    mask = np.zeros(seq_len, dtype=np.uint8)
    for a, b in image_spans:
        mask[a:b] = 1
    r = Request(seq_len, 0, [], budget, window, merge_mode, mask)
    return Workload("tiny", 0, seed, 1, n_q_heads, n_kv_heads, head_dim, False, [r])


# ---------------------------------------------------------------------------------------------
# tensors
# ---------------------------------------------------------------------------------------------

def _gauss_bf16(key: np.uint64, shape: Tuple[int, ...], std: float = 1.0) -> np.ndarray:
    n = int(np.prod(shape))
    return (normal(key, n) * std).astype(np.float32).reshape(shape)


def layer_tensors(w: Workload, layer: int = 0, request: int = 0):
    """Q [L,Hq,d], K [L,Hkv,d], V [L,Hkv,d] of one request and layer as bf16 bit patterns (uint16)."""
    req = w.requests[request]
    L, d = req.seq_len, w.head_dim
    base = (w.seed, w.config_id, layer, request)
    q = _gauss_bf16(stream_key(*base, _T_Q), (L, w.n_q_heads, d))
    v = _gauss_bf16(stream_key(*base, _T_V), (L, w.n_kv_heads, d))
    k = _gauss_bf16(stream_key(*base, _T_K), (L, w.n_kv_heads, d))     # text keys; image noise below
    if req.n_images:
        pos = 0
        for img in range(req.n_images):
            pos += req.segments[img]
            centres = _gauss_bf16(stream_key(*base, _T_CENTRE, img),
                                  (CLUSTERS_PER_IMAGE, w.n_kv_heads, d))
            which = np.arange(IMAGE_TOKENS) // (IMAGE_TOKENS // CLUSTERS_PER_IMAGE)
            k[pos:pos + IMAGE_TOKENS] = centres[which] + np.float32(0.3) * k[pos:pos + IMAGE_TOKENS]
            pos += IMAGE_TOKENS
    if w.k_outliers:
        for h in range(w.n_kv_heads):
            okey = stream_key(w.seed, w.config_id, layer, _T_OUTLIER, h)
            chans: List[int] = []
            i = 0
            while len(chans) < 4:
                c = int(uniform_int(okey, 1, 0, d - 1, offset=i)[0])
                i += 1
                if c not in chans:
                    chans.append(c)
            k[:, h, chans] *= np.float32(8.0)
    return f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v)


def packed_layer_tensors(w: Workload, layer: int = 0):
    """All requests of a layer packed along the token axis, plus the packed mask."""
    qs, ks, vs = zip(*(layer_tensors(w, layer, r) for r in range(len(w.requests))))
    mask = np.concatenate([r.mask for r in w.requests])
    return np.concatenate(qs), np.concatenate(ks), np.concatenate(vs), mask
