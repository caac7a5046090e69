"""Seeded synthetic workloads shaped like the paper's multi-image and long-video prompts.

This module only *generates inputs* (modality span tables, K/V caches, window queries).  It
holds none of the method's arithmetic and is the one module that both the CUDA path's
callers and the CPU oracle's tests may use, so that both sides see the same bits.

Values come from a counter-based generator written with integer tensor ops (a splitmix64
finaliser of seed/layer/tensor/element counters, then Box-Muller), so the same call gives
the same distribution on CPU and on a GPU.  Transcendentals may differ in the last fp32 bit
between devices; parity tests therefore generate once, on one device, and hand the same
bits to both sides.

Real activations, weights and the evaluation suites the paper uses are not reproduced:
these caches only imitate their shapes, modality layout, redundancy (correlated frames)
and per-layer attention density (query temperature).
"""
from __future__ import annotations

import dataclasses
import math

import torch

TEXT = 0
VISUAL = 1

_MASK64 = (1 << 64) - 1


def _splitmix64_int(x: int) -> int:
    x = (x + 0x9E3779B97F4A7C15) & _MASK64
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & _MASK64
    return x ^ (x >> 31)


def _as_i64(x: int) -> int:
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _splitmix64(x: torch.Tensor) -> torch.Tensor:
    x = x + _as_i64(0x9E3779B97F4A7C15)
    x = (x ^ _lsr(x, 30)) * _as_i64(0xBF58476D1CE4E5B9)
    x = (x ^ _lsr(x, 27)) * _as_i64(0x94D049BB133111EB)
    return x ^ _lsr(x, 31)


def stream_key(seed: int, layer: int, tensor_id: int) -> int:
    return _splitmix64_int(_splitmix64_int(seed * 0x10001 + 7) ^ (layer * 0x1000193 + tensor_id * 0x9E37 + 1))


def uniform01(key: int, start: int, count: int, device) -> torch.Tensor:
    """`count` uniforms in (0, 1) for counters start..start+count-1 of stream `key` (fp32)."""
    c = torch.arange(start, start + count, dtype=torch.int64, device=device) + _as_i64(key)
    z = _splitmix64(c)
    return (_lsr(z, 40).to(torch.float32) + 0.5) * (1.0 / (1 << 24))


def normal(key: int, start: int, count: int, device) -> torch.Tensor:
    """`count` standard normals (fp32) for counters start.. of stream `key` (Box-Muller)."""
    c = torch.arange(start, start + count, dtype=torch.int64, device=device) + _as_i64(key)
    z = _splitmix64(c)
    u1 = (_lsr(z, 40).to(torch.float32) + 0.5) * (1.0 / (1 << 24))
    u2 = ((_lsr(z, 16) & 0xFFFFFF).to(torch.float32) + 0.5) * (1.0 / (1 << 24))
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str                      # "f32" or "bf16"
    spans: tuple                    # ((begin, end, modality), ...) sorted, disjoint, covering [0, n)
    window: int
    rho: float                      # global budget as a fraction of L * n
    tau_range: tuple = (0.5, 3.0)   # per-layer query temperature ~ U(lo, hi)
    salient_frac: float = 0.0       # fraction of token positions whose key row is scaled by 3
    frame_tokens: int = 0           # > 0: visual spans are sequences of frames of this many tokens
    frame_rho: float = 0.0          # AR(1) correlation between the same slot of adjacent frames
    visual_offset: float = 0.5      # per-modality mean offset (text offset is 0)
    seed: int = 0
    description: str = ""

    @property
    def n_tokens(self) -> int:
        return self.spans[-1][1]

    @property
    def global_budget(self) -> int:
        return int(round(self.rho * self.n_layers * self.n_tokens))

    @property
    def min_budget(self) -> int:
        return self.window

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def element_size(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def modality(self, device="cpu") -> torch.Tensor:
        m = torch.zeros(self.n_tokens, dtype=torch.uint8, device=device)
        for b, e, mod in self.spans:
            m[b:e] = mod
        return m

    def with_(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def _spans(*parts) -> tuple:
    """parts: (length, modality) in order -> ((begin, end, modality), ...) with neighbours of the
    same modality fused."""
    out, pos = [], 0
    for length, mod in parts:
        if length <= 0:
            continue
        if out and out[-1][2] == mod:
            out[-1] = (out[-1][0], pos + length, mod)
        else:
            out.append((pos, pos + length, mod))
        pos += length
    return tuple(out)


def _tiny() -> Workload:
    return Workload("tiny", 2, 4, 4, 64, "f32",
                    _spans((64, TEXT), (4 * 224, VISUAL), (64, TEXT)), window=64, rho=0.25,
                    salient_frac=0.05, seed=0,
                    description="2 layers, 4 MHA heads, d=64, fp32, 1,024 tokens = 64 text + 4x224 image + 64 text window")


def _multi_image_8k() -> Workload:
    parts = []
    for _ in range(5):
        parts += [(64, TEXT), (1536, VISUAL)]
    parts += [(192, TEXT)]
    return Workload("multi_image_8k", 32, 32, 32, 128, "bf16", _spans(*parts), window=32, rho=0.30,
                    description="LLaVA-NeXT-7B-shaped: 32 layers, 32 MHA heads, d=128, 8,192 tokens = 5 x 1,536 image + 512 text")


def _long_video_19k() -> Workload:
    return Workload("long_video_19k", 28, 28, 4, 128, "bf16",
                    _spans((64, TEXT), (128 * 144, VISUAL), (448, TEXT)), window=32, rho=0.15,
                    salient_frac=0.03, frame_tokens=144, frame_rho=0.9,
                    description="28 layers, 28/4 GQA heads, d=128, 18,944 tokens = 128 frames x 144 + 512 text")


def _multimodal_32k() -> Workload:
    parts = []
    for _ in range(16):
        parts += [(16 * 120, VISUAL), (128, TEXT)]
    return Workload("multimodal_32k", 32, 32, 32, 128, "bf16", _spans(*parts), window=64, rho=0.10,
                    tau_range=(0.3, 4.0), frame_tokens=120,
                    description="32 layers, 32 MHA heads, d=128, 32,768 tokens = 256 frames x 120 + 2,048 interleaved text")


def _long_video_128k() -> Workload:
    return Workload("long_video_128k", 28, 28, 4, 128, "bf16",
                    _spans((48, TEXT), (1000 * 128, VISUAL), (1024, TEXT)), window=32, rho=0.05,
                    salient_frac=0.01, frame_tokens=128, frame_rho=0.95,
                    description="28 layers, 28/4 GQA heads, d=128, 129,072 tokens = 1,000 frames x 128 + 1,072 text")


WORKLOADS = {w.name: w for w in (_tiny(), _multi_image_8k(), _long_video_19k(), _multimodal_32k(), _long_video_128k())}


def small_variant(name: str = "small_gqa", **kw) -> Workload:
    """A reduced shape for fast tests: ragged sizes (no multiple of any tile), GQA, correlated
    frames, salient keys.  Keyword arguments override fields."""
    base = Workload(name, 3, 6, 2, 128, "bf16",
                    _spans((37, TEXT), (9 * 61, VISUAL), (75, TEXT)), window=24, rho=0.2,
                    salient_frac=0.04, frame_tokens=61, frame_rho=0.9, seed=1,
                    description="ragged GQA test shape")
    return base.with_(**kw) if kw else base


def layer_temperature(wl: Workload, layer: int) -> float:
    u = float(uniform01(stream_key(wl.seed, layer, 9), 0, 1, "cpu")[0])
    return wl.tau_range[0] + (wl.tau_range[1] - wl.tau_range[0]) * u


def _cache_tensor(wl: Workload, layer: int, tensor_id: int, device, scale_salient: bool) -> torch.Tensor:
    hkv, n, d = wl.n_kv_heads, wl.n_tokens, wl.head_dim
    key = stream_key(wl.seed, layer, tensor_id)
    out = torch.empty((hkv, n, d), dtype=wl.torch_dtype, device=device)
    mod = wl.modality(device)
    offset = (mod == VISUAL).to(torch.float32)[:, None] * wl.visual_offset
    scale = None
    if scale_salient and wl.salient_frac > 0.0:
        u = uniform01(stream_key(wl.seed, layer, 7), 0, n, device)
        scale = torch.where(u < wl.salient_frac, 3.0, 1.0)[:, None]
    for g in range(hkv):
        z = normal(key, g * n * d, n * d, device).view(n, d)
        if wl.frame_tokens > 0 and wl.frame_rho > 0.0:
            r = wl.frame_rho
            c = math.sqrt(1.0 - r * r)
            for b, e, m in wl.spans:
                if m != VISUAL or (e - b) % wl.frame_tokens != 0:
                    continue
                fr = z[b:e].view((e - b) // wl.frame_tokens, wl.frame_tokens, d)
                for f in range(1, fr.shape[0]):
                    fr[f] = r * fr[f - 1] + c * fr[f]
        z = z + offset
        if scale is not None:
            z = z * scale
        out[g] = z.to(wl.torch_dtype)
    return out


def make_layer(wl: Workload, layer: int, device="cpu"):
    """(q_win [Hq, w, d], k [Hkv, n, d], v [Hkv, n, d]) of one layer in the workload's dtype.

    K, V ~ N(0,1) + visual_offset on visual tokens; frames of a visual span are AR(1)-correlated
    slot by slot; a seeded fraction of token positions (shared by the heads of a layer) has its
    key row scaled by 3 (values unchanged); Q ~ tau_l * N(0,1) with one temperature per layer.
    """
    k = _cache_tensor(wl, layer, 0, device, scale_salient=True)
    v = _cache_tensor(wl, layer, 1, device, scale_salient=False)
    return make_layer_queries(wl, layer, device), k, v


def make_layer_queries(wl: Workload, layer: int, device="cpu"):
    """q_win [Hq, w, d] of make_layer alone."""
    hq, w, d = wl.n_q_heads, wl.window, wl.head_dim
    tau = layer_temperature(wl, layer)
    return (tau * normal(stream_key(wl.seed, layer, 2), 0, hq * w * d, device)).view(hq, w, d).to(wl.torch_dtype)


def make_prompt_queries(wl: Workload, layer: int, device="cpu"):
    """q_all [Hq, n, d] in the workload's dtype: a query row for every prompt token (Eq. 8 without the
    observation-window restriction).  Same distribution as the window's queries; the last `window` rows
    are the rows make_layer returns."""
    hq, n, w, d = wl.n_q_heads, wl.n_tokens, wl.window, wl.head_dim
    tau = layer_temperature(wl, layer)
    q = torch.empty((hq, n, d), dtype=wl.torch_dtype, device=device)
    key = stream_key(wl.seed, layer, 4)
    for h in range(hq):
        q[h] = (tau * normal(key, h * n * d, n * d, device)).view(n, d).to(wl.torch_dtype)
    q[:, n - w:] = make_layer_queries(wl, layer, device)
    return q


def make_visual_queries(wl: Workload, layer: int, n_rows: int, device="cpu"):
    """(q_vis [Hq, n_rows, d] in the workload's dtype, positions int32 [n_rows]): query rows of `n_rows`
    visual tokens spread evenly over the prompt's visual tokens, for the vision-to-text term of the
    cross-modal entropy.  Same distribution as the text window's queries (one temperature per layer)."""
    vis = torch.nonzero(wl.modality("cpu") == VISUAL).flatten()
    if vis.numel() == 0:
        raise ValueError("the workload has no visual token")
    pick = torch.linspace(0, vis.numel() - 1, n_rows).round().to(torch.int64)
    pos = vis[pick].to(torch.int32).to(device)
    hq, d = wl.n_q_heads, wl.head_dim
    tau = layer_temperature(wl, layer)
    q = (tau * normal(stream_key(wl.seed, layer, 3), 0, hq * n_rows * d, device)).view(hq, n_rows, d).to(wl.torch_dtype)
    return q, pos

