"""ctypes front end of the C oracle (``sparsk_oracle.c``).

TEST INFRASTRUCTURE: only tests, the smoke check and the benchmark's CPU-baseline
leg may import this.  It does not import, and is not imported by, the CUDA package.

Weights are passed as NumPy ``uint16`` arrays holding bfloat16 bit patterns:
``embed`` [Vt+Vs, d]; per layer lists ``attn_norm`` [d], ``wq`` [Hq*hd, d], ``wk``,
``wv`` [Hkv*hd, d], ``wo`` [d, Hq*hd], ``mlp_norm`` [d], ``w_gate``, ``w_up`` [F, d],
``w_down`` [d, F], ``head_norm`` [d] or None, ``head_proj`` [Vt+Vs, d] or None.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import build as _build


class _Dims(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads",
                                         "head_dim", "d_ffn", "vocab_text", "vocab_speech")] + [
        ("rms_eps", C.c_double), ("rope_base", C.c_double)] + [
        (n, C.c_int32) for n in ("exit_layer", "refresh_period", "refresh_phase", "text_exit",
                                 "max_len", "text_period", "text_phase", "conf_modalities",
                                 "conf_start")] + [("conf_threshold", C.c_double)]


_PP = C.POINTER(C.c_void_p)


class _Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p)] + [(n, _PP) for n in (
        "attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down",
        "head_norm", "head_proj")]


_PER_LAYER = ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down",
              "head_norm", "head_proj")

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        L.ora_depth.restype = C.c_int32
        L.ora_depth.argtypes = [C.c_int32] * 7
        L.ora_depth_mod.restype = C.c_int32
        L.ora_depth_mod.argtypes = [C.c_int32] * 9
        L.ora_rmsnorm.restype = None
        L.ora_rmsnorm.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_double, C.c_void_p]
        L.ora_rope.restype = None
        L.ora_rope.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_double]
        L.ora_attend.restype = None
        L.ora_attend.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                 C.c_int32, C.c_void_p, C.c_void_p]
        L.ora_model_new.restype = C.c_void_p
        L.ora_model_new.argtypes = [C.POINTER(_Dims), C.POINTER(_Weights)]
        L.ora_model_free.argtypes = [C.c_void_p]
        L.ora_seq_new.restype = C.c_void_p
        L.ora_seq_new.argtypes = [C.c_void_p, C.c_int32]
        L.ora_seq_free.argtypes = [C.c_void_p]
        L.ora_seq_len.restype = C.c_int32
        L.ora_seq_len.argtypes = [C.c_void_p]
        L.ora_seq_pending.restype = C.c_int32
        L.ora_seq_pending.argtypes = [C.c_void_p]
        L.ora_seq_pending_pos.restype = C.c_int32
        L.ora_seq_pending_pos.argtypes = [C.c_void_p, C.c_int32]
        L.ora_get_kv.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        L.ora_set_kv.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        L.ora_set_len.argtypes = [C.c_void_p, C.c_int32]
        L.ora_prefill.restype = C.c_int32
        L.ora_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_int32]
        L.ora_decode_step.restype = C.c_int32
        L.ora_decode_step.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                      C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                      C.POINTER(C.c_double), C.c_void_p, C.c_void_p]
        L.ora_seq_pending_fill.restype = C.c_int32
        L.ora_seq_pending_fill.argtypes = [C.c_void_p, C.c_int32]
        L.ora_entropy.restype = C.c_double
        L.ora_entropy.argtypes = [C.c_void_p, C.c_int32]
        L.ora_decode_step_dyn.restype = C.c_int32
        L.ora_decode_step_dyn.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                          C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                          C.POINTER(C.c_double), C.c_void_p, C.c_void_p, C.c_void_p]
        _lib = L
    return _lib


def depth(modality: int, c: int, K: int, r: int, e: int, L: int, text_exit: int = 0) -> int:
    return lib().ora_depth(modality, c, K, r, e, L, text_exit)


def depth_mod(modality: int, c: int, K_s: int, r_s: int, K_t: int, r_t: int, e: int, L: int,
              text_exit: int) -> int:
    return lib().ora_depth_mod(modality, c, K_s, r_s, K_t, r_t, e, L, text_exit)


def entropy(z) -> float:
    """Entropy (nats) of softmax(z)."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    return lib().ora_entropy(z.ctypes.data, z.size)


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def rmsnorm(x, g_u16, eps):
    x = np.ascontiguousarray(x, dtype=np.float64)
    g = _u16(g_u16)
    y = np.empty_like(x)
    lib().ora_rmsnorm(x.ctypes.data, g.ctypes.data, x.size, eps, y.ctypes.data)
    return y


def rope(x, pos, base):
    x = np.array(x, dtype=np.float64, copy=True)
    lib().ora_rope(x.ctypes.data, x.size, pos, base)
    return x


def attend(q, K, V):
    """q [hd], K/V [n, hd] -> (out [hd], softmax weights [n])."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    K = np.ascontiguousarray(K, dtype=np.float64)
    V = np.ascontiguousarray(V, dtype=np.float64)
    n, hd = K.shape
    w = np.empty(n)
    out = np.empty(hd)
    lib().ora_attend(q.ctypes.data, K.ctypes.data, V.ctypes.data, n, hd, hd, w.ctypes.data,
                     out.ctypes.data)
    return out, w


class OracleModel:
    def __init__(self, dims: dict, weights: dict, max_len: int):
        self.dims = dict(dims)
        self._keep = []
        d = _Dims()
        for k in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn",
                  "vocab_text", "vocab_speech", "exit_layer", "refresh_period", "refresh_phase"):
            setattr(d, k, int(dims[k]))
        d.text_exit = int(dims.get("text_exit", 0))
        d.text_period = int(dims.get("text_period", 0))
        d.text_phase = int(dims.get("text_phase", 0))
        d.conf_modalities = int(dims.get("conf_modalities", 0))
        d.conf_start = int(dims.get("conf_start", 0))
        d.conf_threshold = float(dims.get("conf_threshold", 0.0))
        d.rms_eps = float(dims["rms_eps"])
        d.rope_base = float(dims["rope_base"])
        d.max_len = int(max_len)
        w = _Weights()
        emb = _u16(weights["embed"])
        self._keep.append(emb)
        w.embed = emb.ctypes.data
        nl = d.n_layers
        for name in _PER_LAYER:
            arr = (C.c_void_p * nl)()
            for i in range(nl):
                t = weights[name][i]
                if t is None:
                    arr[i] = None
                else:
                    t = _u16(t)
                    self._keep.append(t)
                    arr[i] = t.ctypes.data
            self._keep.append(arr)
            setattr(w, name, C.cast(arr, _PP))
        self._d, self._w = d, w
        self.V = d.vocab_text + d.vocab_speech
        self.d_model = d.d_model
        self.kv_row = d.n_kv_heads * d.head_dim
        self.max_len = d.max_len
        self._h = lib().ora_model_new(C.byref(d), C.byref(w))
        if not self._h:
            raise ValueError("oracle rejected the dims")

    def new_seq(self, max_pending: int = 64) -> "OracleSeq":
        return OracleSeq(self, max_pending)

    def __del__(self):
        if getattr(self, "_h", None):
            lib().ora_model_free(self._h)
            self._h = None


class OracleSeq:
    def __init__(self, model: OracleModel, max_pending: int):
        self.model = model
        self._h = lib().ora_seq_new(model._h, max_pending)
        if not self._h:
            raise MemoryError("oracle sequence allocation failed")

    def __del__(self):
        if getattr(self, "_h", None):
            lib().ora_seq_free(self._h)
            self._h = None

    @property
    def len(self) -> int:
        return lib().ora_seq_len(self._h)

    @property
    def pending(self) -> list:
        n = lib().ora_seq_pending(self._h)
        return [lib().ora_seq_pending_pos(self._h, j) for j in range(n)]

    @property
    def pending_fill(self) -> list:
        """For each pending position, the layer its K/V is complete up to."""
        n = lib().ora_seq_pending(self._h)
        return [lib().ora_seq_pending_fill(self._h, j) for j in range(n)]

    def get_kv(self, layer: int, pos: int):
        k = np.empty(self.model.kv_row)
        v = np.empty(self.model.kv_row)
        lib().ora_get_kv(self._h, layer, pos, k.ctypes.data, v.ctypes.data)
        return k, v

    def set_kv(self, layer: int, pos: int, k, v):
        k = np.ascontiguousarray(k, dtype=np.float64)
        v = np.ascontiguousarray(v, dtype=np.float64)
        assert k.size == self.model.kv_row and v.size == self.model.kv_row
        lib().ora_set_kv(self._h, layer, pos, k.ctypes.data, v.ctypes.data)

    def set_len(self, n: int):
        lib().ora_set_len(self._h, n)

    def prefill(self, tokens):
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        rc = lib().ora_prefill(self._h, t.ctypes.data, t.size)
        if rc:
            raise RuntimeError(f"oracle prefill failed ({rc})")

    def decode_step(self, token: int, modality: int, counter: int, want_logits: bool = True):
        nt, dp, mg = C.c_int32(), C.c_int32(), C.c_double()
        hid = np.empty(self.model.d_model)
        lg = np.empty(self.model.V) if want_logits else None
        rc = lib().ora_decode_step(self._h, int(token), int(modality), int(counter), C.byref(nt),
                                   C.byref(dp), C.byref(mg), hid.ctypes.data,
                                   lg.ctypes.data if want_logits else None)
        if rc:
            raise RuntimeError(f"oracle decode_step failed ({rc})")
        return {"token": nt.value, "depth": dp.value, "margin": mg.value, "hidden": hid,
                "logits": lg}

    def decode_step_dyn(self, token: int, modality: int, counter: int, forced_depth: int = 0,
                        want_logits: bool = True):
        """A step whose depth is dictated (forced_depth in 1..L) or decided on the way by the
        confidence rule of the dims (forced_depth = 0)."""
        nt, dp, mg = C.c_int32(), C.c_int32(), C.c_double()
        hid = np.empty(self.model.d_model)
        lg = np.empty(self.model.V) if want_logits else None
        ent = np.empty(max(1, self.model.dims["n_layers"] - 1))
        rc = lib().ora_decode_step_dyn(self._h, int(token), int(modality), int(counter), int(forced_depth),
                                       C.byref(nt), C.byref(dp), C.byref(mg), hid.ctypes.data,
                                       lg.ctypes.data if want_logits else None, ent.ctypes.data)
        if rc:
            raise RuntimeError(f"oracle decode_step_dyn failed ({rc})")
        return {"token": nt.value, "depth": dp.value, "margin": mg.value, "hidden": hid,
                "logits": lg, "entropies": ent}
