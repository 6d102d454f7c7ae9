"""Seeded synthetic inputs for the speculative-decoding verify path.

This module only draws random numbers and converts storage formats.  It holds none of
the method's arithmetic (no forward pass, no softmax, no sampling rule), so both the CPU
oracle's tests and the CUDA path's tests may use it without sharing any computation.

Workload shapes follow the paper's setting: a LLaMA-style target attending to a prefix of
projected image embeddings followed by text (Sec. 2.2, Eq. 1), a small LLaMA-style draft
that sees the text only (Sec. 3), block size gamma in {3, 5} (Sec. 4, "Metrics").  The
paper's datasets, tokenizer and trained weights are replaced by draws from N(0, 0.02^2)
(weights), N(0, 1) (image features) and uniform token ids.

Every tensor has its own Philox stream keyed by (seed, tensor tag, layer), so tensors can
be generated lazily, in any order and in parallel with identical results.
"""
from __future__ import annotations

import concurrent.futures as _cf
import os
import zlib
from dataclasses import dataclass, field, asdict

import numpy as np

# ----------------------------------------------------------------------------- formats


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 (round-to-nearest-even); returns the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns to fp32."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------- configs


@dataclass(frozen=True)
class ModelCfg:
    n_layers: int
    d_model: int
    n_heads: int
    d_ffn: int
    vocab: int
    tied_embeddings: bool = False
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    dtype: str = "bf16"  # storage type of weights and KV cache: "bf16" or "fp32"

    @property
    def d_head(self) -> int:
        return self.d_model // self.n_heads

    def n_params(self) -> int:
        d, f, v = self.d_model, self.d_ffn, self.vocab
        emb = v * d if self.tied_embeddings else 2 * v * d
        return self.n_layers * (4 * d * d + 3 * d * f + 2 * d) + emb + d


@dataclass(frozen=True)
class Workload:
    name: str
    target: ModelCfg
    draft: ModelCfg
    n_image: int          # m: image-embedding rows given to the target
    n_prompt: int         # n: prompt token ids
    gamma: int
    n_new: int
    adapter_in: int = 0   # 0: text-only draft; else width of the draft's image features
    draft_mlp: bool = False  # the draft has its own two-layer adapter adapter_in -> d -> d
    seeds: dict = field(default_factory=lambda: {"weights": 1, "inputs": 2, "uniforms": 3})


TINY_TARGET = ModelCfg(2, 256, 4, 688, 1024, False, dtype="fp32")
TINY_DRAFT = ModelCfg(1, 128, 2, 344, 1024, False, dtype="fp32")
LLAVA7B_TARGET = ModelCfg(32, 4096, 32, 11008, 32000, False, dtype="bf16")
DRAFT_115M = ModelCfg(12, 768, 12, 2048, 32000, True, dtype="bf16")
# the draft column of the paper's Table 1: 4 layers, 8 heads, intermediate 2816, hidden 1024
DRAFT_TABLE1 = ModelCfg(4, 1024, 8, 2816, 32000, False, dtype="bf16")


def tiny_workload(gamma: int = 4, adapter: bool = False) -> Workload:
    """The small case: everything the slow CPU implementation finishes in seconds."""
    return Workload("tiny" + ("-adapter" if adapter else ""), TINY_TARGET, TINY_DRAFT, 16, 16,
                    gamma, 32, adapter_in=64 if adapter else 0)


def llava7b_workload(gamma: int = 5, n_layers: int | None = None, adapter: bool = False,
                     n_image: int = 576, n_prompt: int = 64, n_new: int = 256,
                     draft_layers: int | None = None, draft: str = "115m",
                     draft_mlp: bool = False) -> Workload:
    """LLaVA-7B-shaped target with the 115M text-only draft.  ``n_layers`` truncates the
    target (same per-layer shapes) for cases the CPU implementation must finish quickly.
    ``draft="table1"`` selects the draft shape printed in the paper's Table 1; ``draft_mlp``
    gives the draft its own two-layer image adapter 1024 -> d -> d (Appendix A.1)."""
    t = LLAVA7B_TARGET if n_layers is None else ModelCfg(
        n_layers, 4096, 32, 11008, 32000, False, dtype="bf16")
    base = DRAFT_TABLE1 if draft == "table1" else DRAFT_115M
    d = base if draft_layers is None else ModelCfg(
        draft_layers, base.d_model, base.n_heads, base.d_ffn, base.vocab, base.tied_embeddings, dtype="bf16")
    name = "llava7b" if n_layers is None else f"llava7b-{n_layers}L"
    name += "-t1draft" if draft == "table1" else ""
    return Workload(name + ("-adapter" if adapter else "") + ("-mlp" if draft_mlp else ""), t, d, n_image,
                    n_prompt, gamma, n_new, adapter_in=1024 if (adapter or draft_mlp) else 0,
                    draft_mlp=draft_mlp)


# ----------------------------------------------------------------------------- draws


def _rng(seed: int, tag: str, layer: int = 0) -> np.random.Generator:
    key = (int(seed) << 40) ^ (zlib.crc32(tag.encode()) << 8) ^ int(layer)
    return np.random.Generator(np.random.Philox(key=key))


def _normal(seed, tag, layer, shape, std) -> np.ndarray:
    x = _rng(seed, tag, layer).standard_normal(shape, dtype=np.float32)
    x *= np.float32(std)
    return x


def _layer_shapes(cfg: ModelCfg) -> dict:
    d, f = cfg.d_model, cfg.d_ffn
    return {"wq": (d, d), "wk": (d, d), "wv": (d, d), "wo": (d, d),
            "w_gate": (f, d), "w_up": (f, d), "w_down": (d, f)}


class Weights:
    """Weights of one model, each matrix row-major [out, in].

    ``stored[name]`` is what the device library is given: fp32 arrays for an fp32 model,
    bfloat16 bit patterns (uint16) for a bf16 model.  ``f32(name)`` gives the same values
    widened to fp32, which is what the CPU implementation computes with.  Per-layer tensors
    are lists indexed by layer.  Norm gains are 1.0 (fp32), matrices N(0, 0.02^2), no biases.
    """

    def __init__(self, cfg: ModelCfg, seed: int, role: str, adapter_in: int = 0,
                 std: float = 0.02, workers: int | None = None):
        self.cfg, self.seed, self.role = cfg, seed, role
        self.stored: dict = {}
        jobs = [("tok_embed", 0, (cfg.vocab, cfg.d_model))]
        if not cfg.tied_embeddings:
            jobs.append(("lm_head", 0, (cfg.vocab, cfg.d_model)))
        if adapter_in:
            jobs.append(("adapter", 0, (cfg.d_model, adapter_in)))
        for name, shp in _layer_shapes(cfg).items():
            for l in range(cfg.n_layers):
                jobs.append((name, l, shp))

        def make(job):
            name, layer, shp = job
            x = _normal(seed, f"{role}.{name}", layer, shp, std)
            return job, (f32_to_bf16_bits(x) if cfg.dtype == "bf16" else x)

        workers = workers or min(16, os.cpu_count() or 1)
        with _cf.ThreadPoolExecutor(workers) as ex:
            for (name, layer, _), arr in ex.map(make, jobs):
                if name in ("tok_embed", "lm_head", "adapter"):
                    self.stored[name] = arr
                else:
                    self.stored.setdefault(name, [None] * cfg.n_layers)[layer] = arr
        ones = np.ones(cfg.d_model, dtype=np.float32)
        self.stored["attn_norm"] = [ones.copy() for _ in range(cfg.n_layers)]
        self.stored["ffn_norm"] = [ones.copy() for _ in range(cfg.n_layers)]
        self.stored["final_norm"] = ones.copy()
        if cfg.tied_embeddings:
            self.stored["lm_head"] = self.stored["tok_embed"]

    def f32(self, name: str, layer: int | None = None) -> np.ndarray:
        a = self.stored[name] if layer is None else self.stored[name][layer]
        return bf16_bits_to_f32(a) if a.dtype == np.uint16 else a

    # -- several processes on one host (one replica per GPU) share one copy of the stored arrays
    def save(self, directory: str) -> None:
        """Writes every stored array as `<directory>/<name>[.<layer>].npy`."""
        os.makedirs(directory, exist_ok=True)
        for name, a in self.stored.items():
            if name == "lm_head" and self.cfg.tied_embeddings:
                continue
            for layer, arr in (enumerate(a) if isinstance(a, list) else [(None, a)]):
                np.save(os.path.join(directory, name + ("" if layer is None else f".{layer}") + ".npy"), arr)

    @classmethod
    def load(cls, cfg: ModelCfg, seed: int, role: str, directory: str) -> "Weights":
        """The arrays written by `save`, memory-mapped read-only (no second copy in RAM)."""
        self = cls.__new__(cls)
        self.cfg, self.seed, self.role, self.stored = cfg, seed, role, {}
        for fn in sorted(os.listdir(directory)):
            parts = fn[:-4].split(".")
            arr = np.load(os.path.join(directory, fn), mmap_mode="r")
            if len(parts) == 1:
                self.stored[parts[0]] = arr
            else:
                self.stored.setdefault(parts[0], [None] * cfg.n_layers)[int(parts[1])] = arr
        if cfg.tied_embeddings:
            self.stored["lm_head"] = self.stored["tok_embed"]
        return self


def image_embeds(wl: Workload) -> np.ndarray:
    """Projected image embeddings V_1..V_m handed to the target, fp32 [m, d_target].
    N(0,1) for the tiny case, N(0,1)*0.02 for the 7B-shaped case (the scale of its token
    embeddings)."""
    scale = 1.0 if wl.target.d_model < 1024 else 0.02
    return _normal(wl.seeds["inputs"], "image_embeds", 0, (wl.n_image, wl.target.d_model), scale)


def image_features(wl: Workload) -> np.ndarray:
    """Vision-encoder-shaped features H_1..H_m for the draft's adapter, fp32 [m, adapter_in]."""
    return _normal(wl.seeds["inputs"], "image_feats", 0, (wl.n_image, max(wl.adapter_in, 1)), 1.0)


def vision_features(seed: int, m: int, d_in: int) -> np.ndarray:
    """Vision-encoder-shaped features H_1..H_m (CLIP ViT-L/14 gives 576 rows of width 1024),
    fp32 [m, d_in] ~ N(0, 1)."""
    return _normal(seed, f"vision_feats.{d_in}", 0, (m, d_in), 1.0)


def adapter_mlp(seed: int, role: str, d_in: int, d_hid: int, d_out: int, std: float = 0.02):
    """Weights of a two-layer image adapter as bfloat16 bit patterns (uint16), row-major
    [out, in]: W1 [d_hid, d_in], W2 [d_out, d_hid] ~ N(0, std^2), no biases."""
    w1 = _normal(seed, f"{role}.adapter_mlp.w1", 0, (d_hid, d_in), std)
    w2 = _normal(seed, f"{role}.adapter_mlp.w2", 0, (d_out, d_hid), std)
    return f32_to_bf16_bits(w1), f32_to_bf16_bits(w2)


def prompt_ids(wl: Workload) -> np.ndarray:
    g = _rng(wl.seeds["inputs"], "prompt_ids")
    return g.integers(0, wl.target.vocab, size=wl.n_prompt, dtype=np.int32)


def uniforms(seed: int, tag: str, shape) -> np.ndarray:
    """fp32 uniforms in [0, 1) on a 2^-24 grid (so u * 2^24 is an exact integer)."""
    g = _rng(seed, "uniforms." + tag)
    k = g.integers(0, 1 << 24, size=shape, dtype=np.int64)
    return (k.astype(np.float64) / float(1 << 24)).astype(np.float32)


def microbench_logits(B: int, gamma: int, V: int, sigma: float, seed: int = 4):
    """Rejection-sampling microbench inputs: target logits N(0, 3^2) [B, gamma+1, V] and
    draft logits = the first gamma target rows + sigma * N(0,1), both fp32.  sigma sweeps
    the acceptance rate."""
    t = _normal(seed, f"mb.target.{V}.{B}", gamma, (B, gamma + 1, V), 3.0)
    n = _normal(seed, f"mb.noise.{V}.{B}.{sigma}", gamma, (B, gamma, V), sigma)
    return t, (t[:, :gamma, :] + n).astype(np.float32)


def describe(wl: Workload) -> dict:
    d = asdict(wl)
    d["target_params"] = wl.target.n_params()
    d["draft_params"] = wl.draft.n_params()
    return d
