"""Thin ctypes binding of the C ABI in ``include/sparsk.h``.

Argument marshalling only: every step of the decode path runs in the CUDA kernels of
``libsparsk.so``.  PyTorch is used for device memory and streams.  Importing this module
fails loudly if the compiled library is missing; there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsparsk.so")

EXPORTS = ("sparsk_workspace_bytes", "sparsk_create", "sparsk_prefill", "sparsk_decode_step",
           "sparsk_decode_step_host", "sparsk_reset_slot", "sparsk_import_kv", "sparsk_export_kv",
           "sparsk_set_len", "sparsk_slot_state", "sparsk_set_debug", "sparsk_set_option",
           "sparsk_kernel_time", "sparsk_kernel_time_by_class", "sparsk_check", "sparsk_phase_trace", "sparsk_attention", "sparsk_attention_scratch_bytes", "sparsk_attention_static", "sparsk_sampling_scratch_bytes", "sparsk_set_sampling", "sparsk_nucleus_sample",
           "sparsk_launch_count", "sparsk_route_counts", "sparsk_conf_entropies", "sparsk_last_error", "sparsk_destroy")

OK, EINVAL, ECAPACITY, ENOHEAD, ECUDA, ESTATE, ETIMEOUT = 0, -1, -2, -3, -4, -5, -6


class SparskError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"sparsk error {code}: {msg}")
        self.code = code


class Dims(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim",
                                         "d_ffn", "vocab_text", "vocab_speech")] + [
        ("rms_eps", C.c_float), ("rope_base", C.c_float)] + [
        (n, C.c_int32) for n in ("exit_layer", "refresh_period", "refresh_phase", "text_exit",
                                 "max_seqs", "max_seq_len", "max_pending", "prefill_rows",
                                 "text_period", "text_phase", "conf_modalities", "conf_start")] + [
        ("conf_threshold", C.c_float)]


_PP = C.POINTER(C.c_void_p)
PER_LAYER = ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down",
             "head_norm", "head_proj")


class AttnArgs(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("q", "k_cache", "v_cache", "out", "row_slot", "row_pos",
                                          "grp_row0", "grp_nrows")] + [
        (n, C.c_int32) for n in ("n_rows", "n_groups", "max_grp_rows", "max_len", "n_q_heads",
                                 "n_kv_heads", "head_dim", "cache_len", "n_slots")]


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p)] + [(n, _PP) for n in PER_LAYER]


_lib = None


def load():
    """Load ``libsparsk.so`` and declare its signatures.  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2603_09215_b200.build`"
                          " (there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    i32p, u8p, vp = C.POINTER(C.c_int32), C.POINTER(C.c_uint8), C.c_void_p
    L.sparsk_workspace_bytes.restype = C.c_size_t
    L.sparsk_workspace_bytes.argtypes = [C.POINTER(Dims)]
    L.sparsk_create.restype = C.c_int
    L.sparsk_create.argtypes = [C.POINTER(Dims), C.POINTER(Weights), vp, C.c_size_t, vp, C.POINTER(vp)]
    L.sparsk_prefill.restype = C.c_int
    L.sparsk_prefill.argtypes = [vp, C.c_int32, i32p, vp, i32p]
    for name in ("sparsk_decode_step", "sparsk_decode_step_host"):
        f = getattr(L, name)
        f.restype = C.c_int
        f.argtypes = [vp, C.c_int32, i32p, vp, u8p, i32p, vp, vp]
    L.sparsk_reset_slot.restype = C.c_int
    L.sparsk_reset_slot.argtypes = [vp, C.c_int32]
    for name in ("sparsk_import_kv", "sparsk_export_kv"):
        f = getattr(L, name)
        f.restype = C.c_int
        f.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, vp, vp]
    L.sparsk_set_len.restype = C.c_int
    L.sparsk_set_len.argtypes = [vp, C.c_int32, C.c_int32]
    L.sparsk_slot_state.restype = C.c_int
    L.sparsk_slot_state.argtypes = [vp, C.c_int32, i32p, i32p]
    L.sparsk_set_debug.restype = C.c_int
    L.sparsk_set_debug.argtypes = [vp, vp, vp]
    L.sparsk_set_option.restype = C.c_int
    L.sparsk_set_option.argtypes = [vp, C.c_char_p, C.c_int64]
    L.sparsk_kernel_time.restype = C.c_int
    L.sparsk_kernel_time.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    L.sparsk_attention_scratch_bytes.restype = C.c_size_t
    L.sparsk_attention_scratch_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32]
    L.sparsk_attention.restype = C.c_int
    L.sparsk_attention.argtypes = [C.POINTER(AttnArgs), vp, C.c_size_t, vp]
    L.sparsk_attention_static.restype = C.c_int
    L.sparsk_attention_static.argtypes = [C.POINTER(AttnArgs), vp, C.c_char_p, C.c_size_t]
    L.sparsk_sampling_scratch_bytes.restype = C.c_size_t
    L.sparsk_sampling_scratch_bytes.argtypes = [C.POINTER(Dims)]
    L.sparsk_set_sampling.restype = C.c_int
    L.sparsk_set_sampling.argtypes = [vp, C.c_float, C.c_float, vp, vp, C.c_size_t]
    L.sparsk_nucleus_sample.restype = C.c_int
    L.sparsk_nucleus_sample.argtypes = [vp, vp, vp, C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_float, vp, vp]
    L.sparsk_phase_trace.restype = C.c_int
    L.sparsk_phase_trace.argtypes = [vp, C.POINTER(C.c_int64), C.c_int32]
    L.sparsk_kernel_time_by_class.restype = C.c_int
    L.sparsk_kernel_time_by_class.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    L.sparsk_check.restype = C.c_int
    L.sparsk_check.argtypes = [vp]
    L.sparsk_launch_count.restype = C.c_int64
    L.sparsk_launch_count.argtypes = [vp]
    L.sparsk_conf_entropies.restype = C.c_int
    L.sparsk_conf_entropies.argtypes = [vp, C.c_int32, C.POINTER(C.c_float)]
    L.sparsk_route_counts.restype = C.c_int
    L.sparsk_route_counts.argtypes = [vp, C.POINTER(C.c_int64)]
    L.sparsk_last_error.restype = C.c_char_p
    L.sparsk_last_error.argtypes = [vp]
    L.sparsk_destroy.restype = C.c_int
    L.sparsk_destroy.argtypes = [vp]
    _lib = L
    return L


def make_dims(dims: dict, max_seqs: int, max_seq_len: int, max_pending: int, prefill_rows: int = 0) -> Dims:
    d = Dims()
    for k in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab_text",
              "vocab_speech", "exit_layer", "refresh_period", "refresh_phase"):
        setattr(d, k, int(dims[k]))
    d.text_exit = int(dims.get("text_exit", 0))
    d.text_period = int(dims.get("text_period", 0))
    d.text_phase = int(dims.get("text_phase", 0))
    d.conf_modalities = int(dims.get("conf_modalities", 0))
    d.conf_start = int(dims.get("conf_start", 0))
    d.conf_threshold = float(dims.get("conf_threshold", 0.0))
    d.rms_eps = float(dims["rms_eps"])
    d.rope_base = float(dims["rope_base"])
    d.max_seqs, d.max_seq_len, d.max_pending, d.prefill_rows = max_seqs, max_seq_len, max_pending, prefill_rows
    return d


def upload_weights(w: dict, device="cuda") -> dict:
    """NumPy uint16 (bf16 bit patterns) -> torch.bfloat16 tensors on the device."""
    def up(a):
        if a is None:
            return None
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(device).view(torch.bfloat16)
    out = {"embed": up(w["embed"])}
    for name in PER_LAYER:
        out[name] = [up(a) for a in w[name]]
    return out


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def attn_args(q, k_cache, v_cache, out, row_slot, row_pos, grp_row0, grp_nrows, max_grp_rows, max_len,
              n_q_heads) -> AttnArgs:
    """Marshal torch CUDA tensors into the argument block of sparsk_attention.
    q, out: bf16; k_cache / v_cache: [n_slots, n_kv_heads, cache_len, head_dim] float16."""
    assert k_cache.dtype == torch.float16 and v_cache.dtype == torch.float16
    a = AttnArgs()
    a.q, a.k_cache, a.v_cache, a.out = q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), out.data_ptr()
    a.row_slot, a.row_pos = row_slot.data_ptr(), row_pos.data_ptr()
    a.grp_row0, a.grp_nrows = grp_row0.data_ptr(), grp_nrows.data_ptr()
    a.n_rows, a.n_groups = q.shape[0], grp_row0.shape[0]
    a.max_grp_rows, a.max_len = int(max_grp_rows), int(max_len)
    a.n_slots, a.n_kv_heads, a.cache_len, a.head_dim = k_cache.shape
    a.n_q_heads = n_q_heads
    return a


def attention(args: AttnArgs, scratch: torch.Tensor, stream=None) -> int:
    """sparsk_attention on the current (or given) stream; returns the status code."""
    st = (stream or torch.cuda.current_stream()).cuda_stream
    return load().sparsk_attention(C.byref(args), scratch.data_ptr(), scratch.numel(), st)


STATIC_SCRATCH_BYTES = 8 << 20


def attention_static(args: AttnArgs, stream=None):
    """sparsk_attention_static: the attention kernels with the library's built-in scratch area,
    for callers that cannot allocate.  Returns (status code, error text)."""
    st = (stream or torch.cuda.current_stream()).cuda_stream
    buf = C.create_string_buffer(256)
    rc = load().sparsk_attention_static(C.byref(args), st, buf, len(buf))
    return rc, buf.value.decode()


def nucleus_sample(logits: torch.Tensor, uniforms: torch.Tensor, modality: torch.Tensor, vocab_text: int,
                   vocab_speech: int, temperature: float, top_p: float, stream=None) -> torch.Tensor:
    """Tokens [n] (int32, device) drawn from rows of `logits` [n, vocab_text + vocab_speech] (float32)."""
    L = load()
    n = logits.shape[0]
    assert logits.dtype == torch.float32 and logits.is_contiguous() and logits.shape[1] == vocab_text + vocab_speech
    assert uniforms.dtype == torch.float32 and modality.dtype == torch.int32
    out = torch.empty(n, dtype=torch.int32, device=logits.device)
    st = torch.cuda.current_stream().cuda_stream if stream is None else stream
    rc = L.sparsk_nucleus_sample(logits.data_ptr(), uniforms.data_ptr(), modality.data_ptr(), n,
                                 vocab_text, vocab_speech, float(temperature), float(top_p), out.data_ptr(), st)
    if rc != OK:
        raise SparskError(rc, "sparsk_nucleus_sample")
    return out


def attention_scratch_bytes(n_rows: int, n_q_heads: int, head_dim: int) -> int:
    return load().sparsk_attention_scratch_bytes(n_rows, n_q_heads, head_dim)


class Sparsk:
    """One library context.  `weights`: dict of torch.bfloat16 CUDA tensors (see upload_weights)."""

    def __init__(self, dims: dict, weights: dict, max_seqs: int, max_seq_len: int, max_pending: int,
                 prefill_rows: int = 0, stream: torch.cuda.Stream | None = None):
        self.lib = load()
        self.dims = dict(dims)
        self.cd = make_dims(dims, max_seqs, max_seq_len, max_pending, prefill_rows)
        self.V = self.cd.vocab_text + self.cd.vocab_speech
        self.weights = weights                      # keeps the tensors alive
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        nbytes = self.lib.sparsk_workspace_bytes(C.byref(self.cd))
        if nbytes == 0:
            raise SparskError(EINVAL, "invalid dims")
        self.workspace_bytes = nbytes
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=weights["embed"].device)
        cw = Weights()
        cw.embed = weights["embed"].data_ptr()
        self._arrs = []
        for name in PER_LAYER:
            arr = (C.c_void_p * self.cd.n_layers)()
            for i, t in enumerate(weights[name]):
                arr[i] = None if t is None else t.data_ptr()
            self._arrs.append(arr)
            setattr(cw, name, C.cast(arr, _PP))
        h = C.c_void_p()
        rc = self.lib.sparsk_create(C.byref(self.cd), C.byref(cw), self.workspace.data_ptr(), nbytes,
                                    self.stream.cuda_stream, C.byref(h))
        if rc != OK:
            raise SparskError(rc, "sparsk_create failed")
        self.h = h
        self._dbg = None

    # -- helpers
    def _check(self, rc: int):
        if rc != OK:
            raise SparskError(rc, self.lib.sparsk_last_error(self.h).decode())

    def close(self):
        if getattr(self, "h", None):
            self.lib.sparsk_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- C ABI, one method per entry point
    def prefill(self, slots, prompts):
        """prompts: list of int32 arrays (host); copied to the device and ingested."""
        offs = np.zeros(len(prompts) + 1, np.int32)
        offs[1:] = np.cumsum([len(p) for p in prompts])
        cat = np.concatenate([_i32(p) for p in prompts]) if prompts else np.zeros(0, np.int32)
        toks = torch.from_numpy(cat).to(self.workspace.device)
        sl = _i32(slots)
        self._check(self.lib.sparsk_prefill(self.h, len(prompts), sl.ctypes.data_as(C.POINTER(C.c_int32)),
                                            toks.data_ptr(), offs.ctypes.data_as(C.POINTER(C.c_int32))))
        self.stream.synchronize()   # `toks` may be freed after this

    def decode_step(self, slots, token_ids: torch.Tensor, modality, counters, next_tokens: torch.Tensor,
                    exit_depths: torch.Tensor):
        sl, ct = _i32(slots), _i32(counters)
        md = np.ascontiguousarray(modality, dtype=np.uint8)
        self._check(self.lib.sparsk_decode_step(
            self.h, len(sl), sl.ctypes.data_as(C.POINTER(C.c_int32)), token_ids.data_ptr(),
            md.ctypes.data_as(C.POINTER(C.c_uint8)), ct.ctypes.data_as(C.POINTER(C.c_int32)),
            next_tokens.data_ptr(), exit_depths.data_ptr()))

    def decode_step_host(self, slots, token_ids, modality, counters, next_tokens: np.ndarray,
                         exit_depths: np.ndarray):
        sl, ct, tk = _i32(slots), _i32(counters), _i32(token_ids)
        md = np.ascontiguousarray(modality, dtype=np.uint8)
        self._check(self.lib.sparsk_decode_step_host(
            self.h, len(sl), sl.ctypes.data_as(C.POINTER(C.c_int32)), tk.ctypes.data,
            md.ctypes.data_as(C.POINTER(C.c_uint8)), ct.ctypes.data_as(C.POINTER(C.c_int32)),
            next_tokens.ctypes.data, exit_depths.ctypes.data))

    def reset_slot(self, slot: int):
        self._check(self.lib.sparsk_reset_slot(self.h, slot))

    def set_len(self, slot: int, n: int):
        self._check(self.lib.sparsk_set_len(self.h, slot, n))

    def import_kv(self, slot: int, layer: int, first_pos: int, k: torch.Tensor, v: torch.Tensor):
        """k, v: [n, H_kv*hd] float16 on the device (the cache's own element type)."""
        assert k.dtype == torch.float16 and v.dtype == torch.float16 and k.is_contiguous() and v.is_contiguous()
        self._check(self.lib.sparsk_import_kv(self.h, slot, layer, first_pos, k.shape[0], k.data_ptr(),
                                              v.data_ptr()))

    def export_kv(self, slot: int, layer: int, first_pos: int, n: int):
        row = self.cd.n_kv_heads * self.cd.head_dim
        k = torch.empty((n, row), dtype=torch.float16, device=self.workspace.device)
        v = torch.empty_like(k)
        self._check(self.lib.sparsk_export_kv(self.h, slot, layer, first_pos, n, k.data_ptr(), v.data_ptr()))
        return k, v

    def slot_state(self, slot: int):
        a, b = C.c_int32(), C.c_int32()
        self._check(self.lib.sparsk_slot_state(self.h, slot, C.byref(a), C.byref(b)))
        return a.value, b.value

    def set_debug(self, hidden: torch.Tensor | None, logits: torch.Tensor | None):
        self._dbg = (hidden, logits)
        self._check(self.lib.sparsk_set_debug(self.h, None if hidden is None else hidden.data_ptr(),
                                              None if logits is None else logits.data_ptr()))

    def set_sampling(self, temperature: float, top_p: float, uniforms: torch.Tensor | None):
        """Nucleus sampling from now on, with uniforms[i] (float32, device, one per sequence of a
        step) as the random numbers; None goes back to greedy decoding."""
        if uniforms is None:
            self._samp = None
            self._check(self.lib.sparsk_set_sampling(self.h, 0.0, 1.0, None, None, 0))
            return
        assert uniforms.dtype == torch.float32 and uniforms.is_cuda and uniforms.numel() >= self.cd.max_seqs
        nbytes = self.lib.sparsk_sampling_scratch_bytes(C.byref(self.cd))
        old = getattr(self, "_samp", None)
        scratch = old[1] if old else torch.empty(nbytes, dtype=torch.uint8, device=uniforms.device)
        self._samp = (uniforms, scratch)
        self._check(self.lib.sparsk_set_sampling(self.h, float(temperature), float(top_p), uniforms.data_ptr(),
                                                 scratch.data_ptr(), nbytes))

    def set_option(self, name: str, value: int):
        self._check(self.lib.sparsk_set_option(self.h, name.encode(), int(value)))

    def kernel_time(self):
        ms, n = C.c_double(), C.c_int64()
        self._check(self.lib.sparsk_kernel_time(self.h, C.byref(ms), C.byref(n)))
        return ms.value, n.value

    def phase_trace(self, capacity: int = 4096) -> np.ndarray:
        """Nanosecond clock of the persistent kernel's first CTA at its start and after each phase
        of the most recent launch."""
        buf = np.zeros(capacity, np.int64)
        n = self.lib.sparsk_phase_trace(self.h, buf.ctypes.data_as(C.POINTER(C.c_int64)), capacity)
        if n < 0:
            self._check(n)
        return buf[:n]

    def check(self):
        """Synchronise, then raise if a kernel reported a problem through the device status word."""
        self._check(self.lib.sparsk_check(self.h))

    def kernel_time_by_class(self):
        """{class name: (summed ms, launches)} of the launches bracketed since time_kernel was set to 8."""
        ms, n = (C.c_double * 8)(), (C.c_int64 * 8)()
        self._check(self.lib.sparsk_kernel_time_by_class(self.h, ms, n))
        names = ("bookkeeping", "qkv", "attn", "oproj", "gateup", "down", "head", "mega")
        return {k: (ms[i], n[i]) for i, k in enumerate(names)}

    def launch_count(self) -> int:
        return self.lib.sparsk_launch_count(self.h)

    def conf_entropies(self, n_seqs: int) -> np.ndarray:
        """[n_seqs, L] entropies the last decode step saw per layer (column l, -1 where no head was consulted)."""
        L = self.cd.n_layers
        out = np.empty((n_seqs, L), np.float32)
        self._check(self.lib.sparsk_conf_entropies(self.h, n_seqs, out.ctypes.data_as(C.POINTER(C.c_float))))
        return out

    def route_counts(self) -> dict:
        """Layer passes so far by implementation."""
        n = (C.c_int64 * 3)()
        self._check(self.lib.sparsk_route_counts(self.h, n))
        return dict(zip(("mega", "tc", "gemv"), (int(x) for x in n)))
