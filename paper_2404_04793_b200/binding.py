"""ctypes binding of libsq (include/sq.h): same names, argument marshalling only.

Every step of the path runs inside the library's CUDA kernels; PyTorch is used here for
device memory and streams.  There is no fallback: if the shared library is missing or fails
to load, importing a function from it raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_double, c_float, c_int32, c_int64, c_size_t, c_uint8, c_void_p

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("SQ_LIB_PATH") or os.path.join(_PKG, "libsq.so")

SQ_OK, SQ_ERR_INVALID_ARG, SQ_ERR_STATE, SQ_ERR_CAPACITY, SQ_ERR_CUDA, SQ_ERR_UNSUPPORTED = range(6)
SQ_POLICY_SLIDING_WINDOW, SQ_POLICY_STREAMING_LLM, SQ_POLICY_H2O = 0, 1, 2
SQ_F32, SQ_BF16 = 0, 1
SQ_STATIC_SCORE_MAX_ROWS = 1 << 20  # mirrors include/sq.h
_ERR_NAMES = {1: "SQ_ERR_INVALID_ARG", 2: "SQ_ERR_STATE", 3: "SQ_ERR_CAPACITY", 4: "SQ_ERR_CUDA",
              5: "SQ_ERR_UNSUPPORTED"}

# every symbol include/sq.h declares
EXPORTS = ["sq_query_sizes", "sq_ctx_create", "sq_ctx_destroy", "sq_begin_sequence_batch",
           "sq_layer_importance", "sq_layer_importance_fused", "sq_allocate_budgets", "sq_set_budgets", "sq_prefill_compress",
           "sq_decode_step", "sq_evict", "sq_get_cos_sim", "sq_get_budgets", "sq_get_kept", "sq_get_kv",
           "sq_get_len", "sq_status", "sq_last_error", "sq_kv_bytes_per_step", "sq_prompt_scores_static",
           "sq_ctx_export_layout", "sq_ctx_import_layout", "sq_get_importance_state", "sq_set_importance_state"]


class sq_config(ctypes.Structure):
    _fields_ = [(n, c_int32) for n in (
        "n_layer", "n_q_head", "n_kv_head", "head_dim", "hidden", "max_batch", "max_prompt",
        "max_new_tokens", "dtype", "policy", "n_sink", "heavy_num", "heavy_den", "n_cluster", "page_tokens",
        "per_sequence_budgets")]


class sq_layer_layout(ctypes.Structure):
    _fields_ = [(n, c_int64) for n in ("k_off", "v_off", "pos_off", "acc_off", "victim_off")] + \
               [(n, c_int32) for n in ("budget", "cap", "b_heavy", "ring_base", "ring_origin", "n_tok", "n_unit", "reserved")]


class SqError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"{_ERR_NAMES.get(code, code)}: {msg}")
        self.code = code


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libsq.so (building it first if nvcc is available and it is missing)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        from . import build
        build.build_library()
    L = ctypes.CDLL(LIB_PATH)
    P = c_void_p
    L.sq_query_sizes.argtypes = [POINTER(sq_config), c_int64, POINTER(c_size_t), POINTER(c_size_t)]
    L.sq_ctx_create.argtypes = [POINTER(sq_config), c_int64, P, c_size_t, P, c_size_t, POINTER(P)]
    L.sq_ctx_destroy.argtypes = [P]
    L.sq_begin_sequence_batch.argtypes = [P, c_int32, c_int32, P]
    L.sq_layer_importance.argtypes = [P, c_int32, P, P, c_int64, P]
    L.sq_layer_importance_fused.argtypes = [P, c_int32, P, P, P, c_int64, P]
    L.sq_allocate_budgets.argtypes = [P, c_int64, c_double, P]
    L.sq_set_budgets.argtypes = [P, POINTER(c_int32), P]
    L.sq_prefill_compress.argtypes = [P, c_int32, P, P, P, P, P]
    L.sq_decode_step.argtypes = [P, c_int32, c_int32, P, P, P, P, P]
    L.sq_evict.argtypes = [P, c_int32, c_int32, POINTER(c_int32), P]
    L.sq_get_cos_sim.argtypes = [P, POINTER(c_float)]
    L.sq_get_importance_state.argtypes = [P, POINTER(c_double), POINTER(c_int64)]
    L.sq_set_importance_state.argtypes = [P, POINTER(c_double), POINTER(c_int64), P]
    L.sq_get_budgets.argtypes = [P, POINTER(c_int32), POINTER(c_uint8)]
    L.sq_get_kept.argtypes = [P, c_int32, c_int32, c_int32, POINTER(c_int32), POINTER(c_float), POINTER(c_int32)]
    L.sq_get_kv.argtypes = [P, c_int32, c_int32, c_int32, P, P]
    L.sq_get_len.argtypes = [P, c_int32, POINTER(c_int32)]
    L.sq_status.argtypes = [P, POINTER(c_int32)]
    L.sq_last_error.argtypes = [P]
    L.sq_last_error.restype = c_char_p
    L.sq_kv_bytes_per_step.argtypes = [P, c_int32, c_int32, POINTER(c_int64)]
    L.sq_ctx_export_layout.argtypes = [P, POINTER(sq_layer_layout)]
    L.sq_ctx_import_layout.argtypes = [P, POINTER(sq_layer_layout), P]
    L.sq_prompt_scores_static.argtypes = [P, P, c_int32, c_int32, c_int32, c_int32, c_int32, c_int32, P, P]
    for name in EXPORTS:
        if name != "sq_last_error":
            getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


def _dptr(t):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return c_void_p(t.data_ptr())


def _stream():
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def make_config(*, n_layer, n_q_head, n_kv_head, head_dim, hidden, max_batch, max_prompt, max_new_tokens,
                dtype, policy, n_sink=4, heavy_num=1, heavy_den=2, n_cluster=3, page_tokens=16,
                per_sequence_budgets=0) -> sq_config:
    dt = {torch.float32: SQ_F32, torch.bfloat16: SQ_BF16}.get(dtype, dtype)
    return sq_config(n_layer, n_q_head, n_kv_head, head_dim, hidden, max_batch, max_prompt, max_new_tokens,
                     dt, policy, n_sink, heavy_num, heavy_den, n_cluster, page_tokens, int(per_sequence_budgets))


def sq_query_sizes(cfg: sq_config, b_init: int):
    pool, ws = c_size_t(), c_size_t()
    rc = lib().sq_query_sizes(byref(cfg), b_init, byref(pool), byref(ws))
    if rc != SQ_OK:
        raise SqError(rc, "sq_query_sizes")
    return pool.value, ws.value


class Context:
    """One libsq context plus the device memory it lives in (two torch byte tensors).
    Methods carry the C names without the sq_ prefix and take torch CUDA tensors.  With
    per_sequence_budgets the per-layer lists become lists of per-sequence lists ([batch][n_layer])."""

    def __init__(self, cfg: sq_config, b_init: int, device="cuda:0"):
        self.cfg = cfg
        self.b_init = int(b_init)
        self.device = torch.device(device)
        pool_bytes, ws_bytes = sq_query_sizes(cfg, self.b_init)
        with torch.cuda.device(self.device):
            self.pool = torch.empty(pool_bytes + 256, dtype=torch.uint8, device=self.device)
            self.workspace = torch.empty(ws_bytes + 256, dtype=torch.uint8, device=self.device)
            po = (-self.pool.data_ptr()) % 256
            wo = (-self.workspace.data_ptr()) % 256
            h = c_void_p()
            rc = lib().sq_ctx_create(byref(cfg), self.b_init, c_void_p(self.pool.data_ptr() + po), pool_bytes,
                                     c_void_p(self.workspace.data_ptr() + wo), ws_bytes, byref(h))
        if rc != SQ_OK:
            raise SqError(rc, "sq_ctx_create")
        self._h = h
        self.pool_bytes, self.workspace_bytes = pool_bytes, ws_bytes
        self.pool_view = self.pool[po:po + pool_bytes]     # the bytes the library was given

    def close(self):
        if getattr(self, "_h", None):
            lib().sq_ctx_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _ck(self, rc):
        if rc != SQ_OK:
            raise SqError(rc, lib().sq_last_error(self._h).decode())

    def begin_sequence_batch(self, batch, prompt_len):
        self.batch = int(batch)
        self._ck(lib().sq_begin_sequence_batch(self._h, batch, prompt_len, _stream()))

    def layer_importance(self, layer, hidden_in, hidden_out):
        n_tok = hidden_in.numel() // self.cfg.hidden
        self._ck(lib().sq_layer_importance(self._h, layer, _dptr(hidden_in), _dptr(hidden_out), n_tok, _stream()))

    def layer_importance_fused(self, layer, resid, attn_out, hidden_out):
        n_tok = resid.numel() // self.cfg.hidden
        self._ck(lib().sq_layer_importance_fused(self._h, layer, _dptr(resid), _dptr(attn_out), _dptr(hidden_out), n_tok,
                                                 _stream()))

    def allocate_budgets(self, b_init, p):
        self._ck(lib().sq_allocate_budgets(self._h, int(b_init), float(p), _stream()))

    def _rows(self):
        return self.batch if self.cfg.per_sequence_budgets else 1

    def _flatten(self, values, n):
        """[n] -> [n]; with per-sequence budgets [batch][n] -> the C layout (sequence first)."""
        if self.cfg.per_sequence_budgets:
            if len(values) != self.batch or any(not hasattr(v, "__len__") or len(v) != n for v in values):
                raise ValueError("expected one list per sequence")
            return [int(b) for row in values for b in row]
        if len(values) != n:
            raise ValueError("expected one value per layer")
        return [int(b) for b in values]

    def _nest(self, flat, n):
        flat = list(flat)
        if self.cfg.per_sequence_budgets:
            return [flat[s * n:(s + 1) * n] for s in range(self.batch)]
        return flat

    def set_budgets(self, budgets):
        flat = self._flatten(budgets, self.cfg.n_layer)
        arr = (c_int32 * len(flat))(*flat)
        self._ck(lib().sq_set_budgets(self._h, arr, _stream()))

    def prefill_compress(self, layer, k_prompt, v_prompt, q_prompt=None, acc_prompt=None):
        self._ck(lib().sq_prefill_compress(self._h, layer, _dptr(k_prompt), _dptr(v_prompt), _dptr(q_prompt),
                                           _dptr(acc_prompt), _stream()))

    def decode_step(self, layer_begin, layer_end, q, k_new, v_new, out):
        self._ck(lib().sq_decode_step(self._h, layer_begin, layer_end, _dptr(q), _dptr(k_new), _dptr(v_new),
                                      _dptr(out), _stream()))

    def evict(self, layer_begin, layer_end, new_budgets):
        flat = self._flatten(new_budgets, layer_end - layer_begin)
        arr = (c_int32 * len(flat))(*flat)
        self._ck(lib().sq_evict(self._h, layer_begin, layer_end, arr, _stream()))

    def get_importance_state(self):
        """Per-layer sums of cosines and token counts accumulated so far (per-batch budgets)."""
        n = self.cfg.n_layer
        sums, counts = (c_double * n)(), (c_int64 * n)()
        self._ck(lib().sq_get_importance_state(self._h, sums, counts))
        return list(sums), list(counts)

    def set_importance_state(self, sums, counts):
        n = self.cfg.n_layer
        a = (c_double * n)(*[float(x) for x in sums])
        b = (c_int64 * n)(*[int(x) for x in counts])
        self._ck(lib().sq_set_importance_state(self._h, a, b, _stream()))

    def get_cos_sim(self):
        arr = (c_float * (self.cfg.n_layer * self._rows()))()
        self._ck(lib().sq_get_cos_sim(self._h, arr))
        return torch.tensor(self._nest(arr, self.cfg.n_layer), dtype=torch.float32)

    def get_budgets(self):
        n = self.cfg.n_layer * self._rows()
        b = (c_int32 * n)()
        g = (c_uint8 * n)()
        self._ck(lib().sq_get_budgets(self._h, b, g))
        return self._nest(b, self.cfg.n_layer), self._nest([bool(x) for x in g], self.cfg.n_layer)

    def get_len(self, layer):
        n = c_int32()
        self._ck(lib().sq_get_len(self._h, layer, byref(n)))
        return n.value

    def get_kept(self, layer, seq, kv_head):
        cap = self.get_len(layer)
        pos = (c_int32 * max(cap, 1))()
        acc = (c_float * max(cap, 1))()
        n = c_int32()
        self._ck(lib().sq_get_kept(self._h, layer, seq, kv_head, pos, acc, byref(n)))
        return list(pos[: n.value]), list(acc[: n.value])

    def get_kv(self, layer, seq, kv_head):
        cap = self.get_len(layer)                       # the layer's longest unit
        n = len(self.get_kept(layer, seq, kv_head)[0])  # this unit
        dt = torch.float32 if self.cfg.dtype == SQ_F32 else torch.bfloat16
        k = torch.empty(max(cap, 1), self.cfg.head_dim, dtype=dt)
        v = torch.empty(max(cap, 1), self.cfg.head_dim, dtype=dt)
        self._ck(lib().sq_get_kv(self._h, layer, seq, kv_head, c_void_p(k.data_ptr()), c_void_p(v.data_ptr())))
        return k[:n], v[:n]

    def export_layout(self):
        """The cache geometry and fill level per layer (ctypes array, C layout): with a copy of
        `pool` it is the whole state of the batch."""
        arr = (sq_layer_layout * (self.cfg.n_layer * self._rows()))()
        self._ck(lib().sq_ctx_export_layout(self._h, arr))
        return arr

    def import_layout(self, layout):
        self._ck(lib().sq_ctx_import_layout(self._h, layout, _stream()))

    def status(self):
        s = c_int32()
        self._ck(lib().sq_status(self._h, byref(s)))
        return s.value

    def kv_bytes_per_step(self, layer_begin, layer_end):
        b = c_int64()
        self._ck(lib().sq_kv_bytes_per_step(self._h, layer_begin, layer_end, byref(b)))
        return b.value


def sq_prompt_scores_static(q_prompt, k_prompt, acc_out):
    """H2O prompt scores through the entry point that allocates nothing (its intermediate sits
    in a fixed array inside the library).  q_prompt [B, Hq, P, d], k_prompt [B, Hkv, P, d],
    acc_out fp32 [B, Hkv, P]: CUDA tensors the caller already owns.  Raises SqError with
    SQ_ERR_CAPACITY when B * Hq * P exceeds the array."""
    B_, Hq, P_, d = q_prompt.shape
    Hkv = k_prompt.shape[1]
    dt = {torch.float32: SQ_F32, torch.bfloat16: SQ_BF16}[q_prompt.dtype]
    if acc_out.dtype != torch.float32 or tuple(acc_out.shape) != (B_, Hkv, P_):
        raise ValueError("acc_out must be fp32 [batch, n_kv_head, prompt_len]")
    rc = lib().sq_prompt_scores_static(_dptr(q_prompt), _dptr(k_prompt), B_, Hq, Hkv, P_, d, dt, _dptr(acc_out),
                                       _stream())
    if rc != SQ_OK:
        raise SqError(rc, "sq_prompt_scores_static")
