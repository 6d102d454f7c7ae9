"""Thin ctypes binding of the C ABI in include/spd.h (argument marshalling only).

Every step of the path runs in the CUDA library; this module converts numpy arrays and
torch tensors to pointers.  There is no CPU fallback: if libspd.so is missing the import
of any entry point fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspd.so")

SPD_OK, SPD_EINVAL, SPD_ESTATE, SPD_ENOMEM, SPD_EOVERFLOW, SPD_ECUDA, SPD_ETIMEOUT, SPD_ENOTIMPL = range(8)
STATUS_NAMES = ["SPD_OK", "SPD_EINVAL", "SPD_ESTATE", "SPD_ENOMEM", "SPD_EOVERFLOW", "SPD_ECUDA",
                "SPD_ETIMEOUT", "SPD_ENOTIMPL"]

EXPORTS = ["spd_create", "spd_destroy", "spd_fork", "spd_last_error", "spd_prefill", "spd_draft", "spd_verify",
           "spd_generate", "spd_get_logits", "spd_get_draft_logits", "spd_rollback", "spd_get_state",
           "spd_reject_sample", "spd_skinny_gemm", "spd_verify_bytes", "spd_trace",
           "spd_skinny_gemm_noalloc", "spd_image_adapter", "spd_truncate_probs", "spd_skinny_gemm_status",
           "spd_wait_selftest", "spd_draft_tree", "spd_verify_tree", "spd_batch_create", "spd_batch_destroy",
           "spd_batch_draft", "spd_batch_verify", "spd_batch_get_logits", "spd_batch_verify_bytes"]


class SpdError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"{STATUS_NAMES[status] if 0 <= status < 8 else status}: {msg}")
        self.status = status


class ModelCfgC(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("d_model", C.c_int), ("n_heads", C.c_int), ("d_ffn", C.c_int),
                ("vocab", C.c_int), ("tied_embeddings", C.c_int), ("rms_eps", C.c_float),
                ("rope_theta", C.c_float), ("dtype", C.c_int)]


class CfgC(C.Structure):
    _fields_ = [("target", ModelCfgC), ("draft", ModelCfgC), ("max_seq", C.c_int), ("gamma_max", C.c_int),
                ("temperature", C.c_float), ("greedy", C.c_int), ("draft_adapter_in", C.c_int),
                ("stream", C.c_void_p), ("grid_mode", C.c_int), ("top_k", C.c_int), ("top_p", C.c_float)]


_PP = C.POINTER(C.c_void_p)


class WeightsC(C.Structure):
    _fields_ = [("tok_embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("adapter", C.c_void_p), ("attn_norm", _PP), ("wq", _PP), ("wk", _PP), ("wv", _PP),
                ("wo", _PP), ("ffn_norm", _PP), ("w_gate", _PP), ("w_up", _PP), ("w_down", _PP)]


class StatsC(C.Structure):
    _fields_ = [("blocks", C.c_int), ("accepted", C.c_int), ("tokens", C.c_int), ("tau", C.c_float),
                ("ms_total", C.c_float), ("ms_draft", C.c_float), ("ms_verify", C.c_float),
                ("graph_replays", C.c_int)]


_lib = None


def lib() -> C.CDLL:
    """The loaded library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with "
                              "`python -m paper_2404_08856_b200.build` (needs nvcc); "
                              "there is no CPU fallback")
        _lib = C.CDLL(LIB_PATH)
        _lib.spd_last_error.restype = C.c_char_p
        _lib.spd_last_error.argtypes = [C.c_void_p]
        _lib.spd_destroy.restype = None
        _lib.spd_destroy.argtypes = [C.c_void_p]
        _lib.spd_batch_destroy.restype = None
        _lib.spd_batch_destroy.argtypes = [C.c_void_p]
        for name in EXPORTS:
            if name not in ("spd_last_error", "spd_destroy", "spd_batch_destroy"):
                getattr(_lib, name).restype = C.c_int
    return _lib


def _ptr(a) -> C.c_void_p:
    """Pointer of a numpy array (host) or of anything with data_ptr() (torch tensor)."""
    if a is None:
        return C.c_void_p(0)
    if hasattr(a, "data_ptr"):
        return C.c_void_p(a.data_ptr())
    assert a.flags["C_CONTIGUOUS"]
    return C.c_void_p(a.ctypes.data)


def model_cfg_c(cfg) -> ModelCfgC:
    return ModelCfgC(cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.d_ffn, cfg.vocab,
                     int(cfg.tied_embeddings), cfg.rms_eps, cfg.rope_theta, 1 if cfg.dtype == "bf16" else 0)


def weights_c(stored: dict, n_layers: int):
    """`stored`: name -> array, per-layer names -> list of arrays (host numpy or device
    tensors).  Returns (struct, keepalive)."""
    keep = []

    def arr(name):
        a = (C.c_void_p * n_layers)(*[_ptr(x).value for x in stored[name]])
        keep.append(a)
        return C.cast(a, _PP)

    w = WeightsC(_ptr(stored["tok_embed"]), _ptr(stored.get("lm_head")), _ptr(stored["final_norm"]),
                 _ptr(stored.get("adapter")), arr("attn_norm"), arr("wq"), arr("wk"), arr("wv"), arr("wo"),
                 arr("ffn_norm"), arr("w_gate"), arr("w_up"), arr("w_down"))
    keep.append(stored)
    return w, keep


class Spd:
    """One speculative-decoding context (one sequence) on the current CUDA device."""

    def __init__(self, target_cfg, draft_cfg, target_stored: dict, draft_stored: dict, max_seq: int,
                 gamma_max: int, temperature: float = 1.0, greedy: bool = False, adapter_in: int = 0,
                 stream: int = 0, grid_mode: int = 0, top_k: int = 0, top_p: float = 0.0):
        L = lib()
        self.vocab = target_cfg.vocab
        self.greedy = greedy
        cfg = CfgC(model_cfg_c(target_cfg), model_cfg_c(draft_cfg), max_seq, gamma_max, temperature,
                   int(greedy), adapter_in, C.c_void_p(stream), int(grid_mode), int(top_k), float(top_p))
        tw, k1 = weights_c(target_stored, target_cfg.n_layers)
        dw, k2 = weights_c(draft_stored, draft_cfg.n_layers)
        self._ctx = C.c_void_p(0)
        st = L.spd_create(C.byref(tw), C.byref(dw), C.byref(cfg), C.byref(self._ctx))
        del k1, k2
        if st != SPD_OK:
            raise SpdError(st, "spd_create failed (see stderr)")

    def _check(self, st: int):
        if st != SPD_OK:
            raise SpdError(st, lib().spd_last_error(self._ctx).decode())

    def fork(self) -> "Spd":
        """Another sequence on the same weights (see spd_fork): own KV caches and state."""
        other = object.__new__(Spd)
        other.vocab, other.greedy = self.vocab, self.greedy
        other._ctx = C.c_void_p(0)
        self._check(lib().spd_fork(self._ctx, C.byref(other._ctx)))
        return other

    def close(self):
        if getattr(self, "_ctx", None) and self._ctx.value:
            lib().spd_destroy(self._ctx)
            self._ctx = C.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def prefill(self, image_embeds, prompt_ids, u0=None, draft_image_feats=None) -> int:
        m = 0 if image_embeds is None else int(image_embeds.shape[0])
        ids = np.ascontiguousarray(prompt_ids, dtype=np.int32) if not hasattr(prompt_ids, "data_ptr") else prompt_ids
        first = C.c_int32(0)
        u = None if u0 is None else C.byref(C.c_float(float(u0)))
        self._check(lib().spd_prefill(self._ctx, _ptr(image_embeds), m, _ptr(draft_image_feats), _ptr(ids),
                                      int(ids.shape[0]), u, C.byref(first)))
        return first.value

    def image_adapter(self, feats, w1, w2, out):
        """out[m, d_out] = GELU(feats[m, d_in] w1[d_hid, d_in]^T) w2[d_out, d_hid]^T (see
        spd_image_adapter): w1, w2 bf16 device tensors, out an fp32 device tensor."""
        self._check(lib().spd_image_adapter(self._ctx, _ptr(feats), int(feats.shape[0]), int(feats.shape[1]),
                                            _ptr(w1), int(w1.shape[0]), _ptr(w2), int(w2.shape[0]), _ptr(out)))
        return out

    def draft(self, gamma: int, uniforms=None, probs_out=None):
        ids = np.zeros(gamma, dtype=np.int32)
        u = None if uniforms is None else np.ascontiguousarray(uniforms, dtype=np.float32)
        self._check(lib().spd_draft(self._ctx, gamma, _ptr(u), _ptr(ids), _ptr(probs_out)))
        return ids

    def verify(self, gamma: int, uniforms=None, draft_ids=None, draft_probs=None):
        u = None if uniforms is None else np.ascontiguousarray(uniforms, dtype=np.float32)
        ids = draft_ids if (draft_ids is None or hasattr(draft_ids, "data_ptr")) \
            else np.ascontiguousarray(draft_ids, dtype=np.int32)
        a, nxt = C.c_int32(0), C.c_int32(0)
        self._check(lib().spd_verify(self._ctx, gamma, _ptr(ids), _ptr(draft_probs), _ptr(u), C.byref(a),
                                     C.byref(nxt)))
        return a.value, nxt.value

    def draft_tree(self, branching, uniforms=None, probs_out=None):
        """See spd_draft_tree.  Returns (parent [n+1], node ids [n])."""
        br = np.ascontiguousarray(branching, dtype=np.int32)
        n, lvl = 0, 1
        for b in br:
            lvl *= int(b)
            n += lvl
        ids = np.zeros(max(n, 1), dtype=np.int32)
        parent = np.zeros(max(n, 1) + 1, dtype=np.int32)
        u = None if uniforms is None else np.ascontiguousarray(uniforms, dtype=np.float32)
        self._check(lib().spd_draft_tree(self._ctx, len(br), _ptr(br), _ptr(u), _ptr(ids), _ptr(parent),
                                         _ptr(probs_out)))
        return parent[: n + 1], ids[:n]

    def verify_tree(self, parent, uniforms=None, node_ids=None, draft_probs=None):
        """See spd_verify_tree.  Returns (path, next_token)."""
        par = np.ascontiguousarray(parent, dtype=np.int32)
        n = len(par) - 1
        u = None if uniforms is None else np.ascontiguousarray(uniforms, dtype=np.float32)
        ids = node_ids if (node_ids is None or hasattr(node_ids, "data_ptr")) \
            else np.ascontiguousarray(node_ids, dtype=np.int32)
        a, nxt = C.c_int32(0), C.c_int32(0)
        path = np.zeros(8, dtype=np.int32)
        self._check(lib().spd_verify_tree(self._ctx, n, _ptr(par), _ptr(ids), _ptr(draft_probs), _ptr(u),
                                          C.byref(a), _ptr(path), C.byref(nxt)))
        return [int(x) for x in path[: a.value]], nxt.value

    def draft_async(self, gamma: int, uniforms_dev=None):
        """Enqueue gamma draft steps with device-resident uniforms; nothing is read back."""
        self._check(lib().spd_draft(self._ctx, gamma, _ptr(uniforms_dev), None, None))

    def verify_async(self, gamma: int, uniforms_dev=None):
        """Enqueue a verify step with device-resident uniforms; nothing is read back."""
        self._check(lib().spd_verify(self._ctx, gamma, None, None, _ptr(uniforms_dev), None, None))

    def generate(self, n_new: int, gamma: int, uniforms=None):
        out = np.zeros(n_new, dtype=np.int32)
        st = StatsC()
        u = None if uniforms is None else (uniforms if hasattr(uniforms, "data_ptr")
                                           else np.ascontiguousarray(uniforms, dtype=np.float32))
        self._check(lib().spd_generate(self._ctx, n_new, gamma, _ptr(u), _ptr(out), C.byref(st)))
        return out, {"blocks": st.blocks, "accepted": st.accepted, "tokens": st.tokens, "tau": st.tau,
                     "ms_total": st.ms_total, "ms_draft": st.ms_draft, "ms_verify": st.ms_verify,
                     "graph_replays": st.graph_replays}

    def get_logits(self, rows: int) -> np.ndarray:
        out = np.zeros((rows, self.vocab), dtype=np.float32)
        self._check(lib().spd_get_logits(self._ctx, _ptr(out), rows))
        return out

    def get_draft_logits(self, rows: int) -> np.ndarray:
        out = np.zeros((rows, self.vocab), dtype=np.float32)
        self._check(lib().spd_get_draft_logits(self._ctx, _ptr(out), rows))
        return out

    def rollback(self, n_text: int, prev_token: int, pending_token: int):
        self._check(lib().spd_rollback(self._ctx, n_text, prev_token, pending_token))

    def get_state(self):
        n, p = C.c_int32(0), C.c_int32(0)
        self._check(lib().spd_get_state(self._ctx, C.byref(n), C.byref(p)))
        return n.value, p.value

    def trace(self) -> np.ndarray:
        """Phase timestamps (ns) of the last verify step; the first call enables tracing."""
        out = np.zeros(1024, dtype=np.uint64)
        n = C.c_int(0)
        self._check(lib().spd_trace(self._ctx, _ptr(out), 1024, C.byref(n)))
        return out[: n.value].copy()

    def wait_selftest(self, which: int, polls: int = 2000) -> int:
        """Runs a bounded device-side wait that cannot succeed (see spd_wait_selftest) and returns
        the status the library reports for it (SPD_ETIMEOUT when the give-up path works)."""
        return int(lib().spd_wait_selftest(self._ctx, int(which), C.c_uint(polls)))

    def verify_bytes(self, gamma: int) -> float:
        b = C.c_double(0)
        self._check(lib().spd_verify_bytes(self._ctx, gamma, C.byref(b)))
        return b.value


class SpdBatch:
    """Several sequences (contexts that share their weights) decoded with one pass over the weights
    per step; see spd_batch_create."""

    def __init__(self, seqs):
        self.seqs = list(seqs)
        self.B = len(self.seqs)
        arr = (C.c_void_p * self.B)(*[s._ctx.value for s in self.seqs])
        self._bt = C.c_void_p(0)
        st = lib().spd_batch_create(arr, self.B, C.byref(self._bt))
        if st != SPD_OK:
            raise SpdError(st, lib().spd_last_error(self.seqs[0]._ctx).decode())

    def _check(self, st: int):
        if st != SPD_OK:
            raise SpdError(st, lib().spd_last_error(self.seqs[0]._ctx).decode())

    def close(self):
        if getattr(self, "_bt", None) and self._bt.value:
            lib().spd_batch_destroy(self._bt)
            self._bt = C.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def draft(self, gamma: int, uniforms=None, read_ids: bool = True):
        """uniforms [B, gamma] (numpy or device tensor).  Returns ids [B, gamma] (or None)."""
        u = uniforms if (uniforms is None or hasattr(uniforms, "data_ptr")) \
            else np.ascontiguousarray(uniforms, dtype=np.float32)
        ids = np.zeros((self.B, gamma), dtype=np.int32) if read_ids else None
        self._check(lib().spd_batch_draft(self._bt, gamma, _ptr(u), _ptr(ids)))
        return ids

    def verify(self, gamma: int, uniforms=None, read: bool = True):
        """uniforms [B, gamma+1].  Returns (n_accepted [B], next_token [B]) (or None)."""
        u = uniforms if (uniforms is None or hasattr(uniforms, "data_ptr")) \
            else np.ascontiguousarray(uniforms, dtype=np.float32)
        a = np.zeros(self.B, dtype=np.int32) if read else None
        n = np.zeros(self.B, dtype=np.int32) if read else None
        self._check(lib().spd_batch_verify(self._bt, gamma, _ptr(u), _ptr(a), _ptr(n)))
        return (a, n) if read else None

    def get_logits(self, rows: int) -> np.ndarray:
        out = np.zeros((rows, self.seqs[0].vocab), dtype=np.float32)
        self._check(lib().spd_batch_get_logits(self._bt, _ptr(out), rows))
        return out

    def verify_bytes(self, gamma: int) -> float:
        b = C.c_double(0)
        self._check(lib().spd_batch_verify_bytes(self._bt, gamma, C.byref(b)))
        return b.value


def reject_sample(p, q, ids, u, gamma: int, greedy: bool, n_acc, nxt, stream: int = 0):
    """Device tensors in, device tensors out (see spd_reject_sample)."""
    B, V = int(p.shape[0]), int(p.shape[-1])
    st = lib().spd_reject_sample(_ptr(p), _ptr(q), _ptr(ids), _ptr(u), B, gamma, V, int(greedy), _ptr(n_acc),
                                 _ptr(nxt), C.c_void_p(stream))
    if st != SPD_OK:
        raise SpdError(st, "spd_reject_sample")


def truncate_probs(probs, out, top_k: int = 0, top_p: float = 1.0, stream: int = 0):
    """Top-k / top-p truncation and renormalisation of fp32 probability rows on the device
    (see spd_truncate_probs); `out` may be `probs`."""
    V = int(probs.shape[-1])
    rows = int(probs.numel() // V)
    st = lib().spd_truncate_probs(_ptr(probs), _ptr(out), rows, V, int(top_k), C.c_float(top_p), C.c_void_p(stream))
    if st != SPD_OK:
        raise SpdError(st, "spd_truncate_probs")


def skinny_gemm(x, w, y, dtype: int, stream: int = 0):
    """y[M,N] = x[M,K] w[N,K]^T on device tensors (see spd_skinny_gemm)."""
    M, K = int(x.shape[0]), int(x.shape[1])
    N = int(w.shape[0])
    st = lib().spd_skinny_gemm(_ptr(x), _ptr(w), dtype, M, N, K, _ptr(y), C.c_void_p(stream))
    if st != SPD_OK:
        raise SpdError(st, "spd_skinny_gemm")


def skinny_gemm_status(noalloc: bool, stream: int = 0) -> int:
    """Status of the last stand-alone GEMM call on the current device (see spd_skinny_gemm_status)."""
    return int(lib().spd_skinny_gemm_status(int(noalloc), C.c_void_p(stream)))


NOALLOC_MAX_PACKED_BYTES = 16 << 20


def skinny_gemm_noalloc(x, w, y, dtype: int, stream: int = 0):
    """y[M,N] = x[M,K] w[N,K]^T on device tensors through the entry point that never
    allocates device memory (fixed scratch inside the library; see spd_skinny_gemm_noalloc).
    Raises SpdError(SPD_EOVERFLOW) when the repacked weights exceed the fixed scratch."""
    M, K = int(x.shape[0]), int(x.shape[1])
    N = int(w.shape[0])
    st = lib().spd_skinny_gemm_noalloc(_ptr(x), _ptr(w), dtype, M, N, K, _ptr(y), C.c_void_p(stream))
    if st != SPD_OK:
        raise SpdError(st, "spd_skinny_gemm_noalloc")
