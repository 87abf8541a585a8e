"""ctypes binding of libgram.so: the same names as include/gram.h, argument marshalling only.

Device buffers are torch CUDA tensors (torch is used for device memory and
streams, nothing else); every step of the path runs inside the library.  The
library is loaded on first use and a missing libgram.so is an error: there is
no fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgram.so")

GRAM_F32, GRAM_BF16 = 0, 1
GRAM_POOL_MEAN, GRAM_POOL_CLS, GRAM_POOL_ADDITIVE = 0, 1, 2
GRAM_TASK_NONE, GRAM_TASK_KT, GRAM_TASK_NR = 0, 1, 2
GRAM_MODULE_CE, GRAM_MODULE_TASK = 0, 1
GRAM_OPT_SGD, GRAM_OPT_ADAM = 0, 1
GRAM_MULTI_TABLE, GRAM_MULTI_PSEUDO_TARGET = 0, 1
STATUS = {0: "GRAM_OK", 1: "GRAM_ERR_ARG", 2: "GRAM_ERR_ID_RANGE", 3: "GRAM_ERR_WORKSPACE", 4: "GRAM_ERR_UNSUPPORTED",
          5: "GRAM_ERR_CUDA", 6: "GRAM_ERR_TIMEOUT"}

# every symbol include/gram.h declares
SYMBOLS = ["gram_create", "gram_destroy", "gram_sync", "gram_last_error", "gram_param_count", "gram_set_params",
           "gram_get_params", "gram_get_grads", "gram_zero_grads", "gram_set_item_tokens", "gram_set_item_lengths",
           "gram_dedup",
           "gram_encode_unique", "gram_gather", "gram_accumulate", "gram_accumulate_multistep", "gram_touched_list",
           "gram_task", "gram_encoder_backward", "gram_step", "gram_step_host", "gram_cache_fill",
           "gram_window_reset", "gram_get_window", "gram_gemm_bf16", "gram_profile", "gram_profile_read",
           "gram_launch_count", "gram_profile_dump", "gram_accumulate_static", "gram_optimizer_step",
           "gram_optimizer_reset", "gram_noam_rate", "gram_adam_update", "gram_state_export", "gram_state_import",
           "gram_optimizer_export", "gram_optimizer_import", "gram_selftest_bounded_wait", "gram_grads_device",
           "gram_gemm_bf16_epilogue"]

KINDS = ["gemm", "attention", "layernorm", "colsum", "embed_pool", "dedup", "gather", "accumulate", "task_head", "other",
         "optimizer"]


class GramConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("dtype", "n_items", "l_t", "vocab", "d", "n_heads", "d_ff", "n_layers",
                                          "pooling", "task", "task_layers", "task_heads", "task_d_ff",
                                          "task_attn_only", "d_a", "n_cand", "B_max", "L")] + \
               [("P_max", C.c_int64), ("d_max", C.c_int32), ("K", C.c_int32), ("ce_micro_batch", C.c_int32),
                ("lr_task", C.c_float), ("lr_ce", C.c_float), ("optimizer", C.c_int32), ("noam_warmup", C.c_int32),
                ("adam_beta1", C.c_float), ("adam_beta2", C.c_float), ("adam_eps", C.c_float),
                ("multistep_variant", C.c_int32), ("refresh_after_update", C.c_int32), ("defer_update", C.c_int32)]


class GramGemmEpilogue(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("d_bias", "d_res", "d_res_mean", "d_res_rstd", "d_res_gamma", "d_res_beta",
                                          "d_gelu_grad_out", "d_gelu_grad_in", "d_copy_bf16")] + \
               [("gelu", C.c_int32), ("accumulate", C.c_int32)]


class GramStepReport(C.Structure):
    _fields_ = [("loss", C.c_float), ("n_positions", C.c_int32), ("n_unique", C.c_int32), ("boost_ratio", C.c_float),
                ("n_touched", C.c_int32), ("encoder_pass", C.c_int32), ("n_encoded", C.c_int32),
                ("ms_dedup", C.c_float), ("ms_encode", C.c_float), ("ms_gather", C.c_float), ("ms_task", C.c_float),
                ("ms_accumulate", C.c_float), ("ms_backward", C.c_float), ("ms_total", C.c_float)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class GramError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"{STATUS.get(status, status)}: {msg}")
        self.status = status


_lib = None


def lib():
    """The loaded library; raises if libgram.so has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} is missing: build it with `python -m paper_2204_04179_b200.build` "
                                    "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        for s in SYMBOLS:
            getattr(L, s).restype = C.c_int
        L.gram_last_error.restype = C.c_char_p
        _lib = L
    return _lib


def noam_rate(t: int, peak: float, warmup: int) -> float:
    """The library's host-side learning-rate curve (no GPU needed)."""
    out = C.c_float(0)
    st = lib().gram_noam_rate(C.c_int64(int(t)), C.c_float(peak), C.c_int32(int(warmup)), C.byref(out))
    if st != 0:
        raise GramError(st, "gram_noam_rate")
    return out.value


def config_from_shape(shape, **over) -> GramConfig:
    """GramConfig of a synth.GramShape."""
    cfg = GramConfig()
    cfg.dtype = GRAM_BF16 if shape.dtype == "bf16" else GRAM_F32
    for k in ("n_items", "l_t", "vocab", "d", "n_heads", "d_ff", "n_layers", "task_layers", "task_heads", "task_d_ff",
              "d_a", "n_cand", "L", "K"):
        setattr(cfg, k, int(getattr(shape, k)))
    cfg.pooling = {"mean": GRAM_POOL_MEAN, "cls": GRAM_POOL_CLS, "additive": GRAM_POOL_ADDITIVE}[shape.pooling]
    cfg.task = {"kt": GRAM_TASK_KT, "nr": GRAM_TASK_NR}[shape.task]
    cfg.task_attn_only = int(shape.task_attn_only)
    cfg.B_max = int(shape.B)
    for k, v in over.items():
        setattr(cfg, k, v)
    return cfg


def _ptr(t) -> C.c_void_p:
    """Device (or host) address of a torch tensor / numpy array; None -> NULL."""
    if t is None:
        return C.c_void_p(0)
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return C.c_void_p(t.ctypes.data)
    assert t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


class Gram:
    """One library context.  Methods mirror the C calls one to one."""

    def __init__(self, cfg: GramConfig):
        self.cfg = cfg
        self._h = C.c_void_p(0)
        st = lib().gram_create(C.byref(cfg), C.byref(self._h))
        if st != 0:
            raise GramError(st, "gram_create failed (see stderr)")

    def close(self):
        if self._h:
            lib().gram_destroy(self._h)
            self._h = C.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _ck(self, st: int):
        if st != 0:
            raise GramError(st, lib().gram_last_error(self._h).decode())

    def sync(self, stream=None):
        self._ck(lib().gram_sync(self._h, _stream(stream)))

    # parameters
    def param_count(self, module: int) -> int:
        n = C.c_size_t(0)
        self._ck(lib().gram_param_count(self._h, module, C.byref(n)))
        return n.value

    def set_params(self, module: int, flat: np.ndarray):
        flat = np.ascontiguousarray(flat, dtype=np.float32)
        self._ck(lib().gram_set_params(self._h, module, _ptr(flat), C.c_size_t(flat.size)))

    def get_params(self, module: int) -> np.ndarray:
        out = np.empty(self.param_count(module), np.float32)
        self._ck(lib().gram_get_params(self._h, module, _ptr(out), C.c_size_t(out.size)))
        return out

    def get_grads(self, module: int) -> np.ndarray:
        out = np.empty(self.param_count(module), np.float32)
        self._ck(lib().gram_get_grads(self._h, module, _ptr(out), C.c_size_t(out.size)))
        return out

    def grads_device(self, module: int):
        """(device address, element count) of a module's fp32 gradient buffer."""
        p, n = C.c_void_p(0), C.c_size_t(0)
        self._ck(lib().gram_grads_device(self._h, module, C.byref(p), C.byref(n)))
        return p.value or 0, n.value

    def zero_grads(self, module: int, stream=None):
        self._ck(lib().gram_zero_grads(self._h, module, _stream(stream)))

    def optimizer_step(self, module: int, stream=None):
        self._ck(lib().gram_optimizer_step(self._h, module, _stream(stream)))

    def optimizer_reset(self, stream=None):
        self._ck(lib().gram_optimizer_reset(self._h, _stream(stream)))

    def adam_update(self, w, g, m, v, t, rate, beta1=0.9, beta2=0.999, eps=1e-8, w_bf16=None, stream=None):
        self._ck(lib().gram_adam_update(self._h, _ptr(w), _ptr(g), _ptr(m), _ptr(v), C.c_size_t(w.numel()), C.c_int64(int(t)),
                                        C.c_float(rate), C.c_float(beta1), C.c_float(beta2), C.c_float(eps), _ptr(w_bf16),
                                        _stream(stream)))

    def set_item_tokens(self, tokens: np.ndarray):
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        self._ck(lib().gram_set_item_tokens(self._h, _ptr(tokens)))

    def set_item_lengths(self, lengths: Optional[np.ndarray]):
        if lengths is None:
            self._ck(lib().gram_set_item_lengths(self._h, C.c_void_p(0)))
            return
        lengths = np.ascontiguousarray(lengths, dtype=np.int32)
        assert lengths.size == self.cfg.n_items
        self._ck(lib().gram_set_item_lengths(self._h, _ptr(lengths)))

    def selftest_bounded_wait(self, stream=None):
        """Queues a wait that nothing satisfies; the next sync() raises GramError with status GRAM_ERR_TIMEOUT."""
        self._ck(lib().gram_selftest_bounded_wait(self._h, _stream(stream)))

    # stages
    def dedup(self, ids, n_items, unique, inverse, perm, seg_off, n_unique, stream=None):
        self._ck(lib().gram_dedup(self._h, _ptr(ids), C.c_int64(ids.numel()), C.c_int32(n_items), _ptr(unique),
                                  _ptr(inverse), _ptr(perm), _ptr(seg_off), _ptr(n_unique), _stream(stream)))

    def encode_unique(self, item_tokens, items, U, H, save_activations=False, stream=None):
        self._ck(lib().gram_encode_unique(self._h, _ptr(item_tokens), _ptr(items), C.c_int32(U), _ptr(H),
                                          C.c_int(int(save_activations)), _stream(stream)))

    def gather(self, src, index, E, P=None, stream=None):
        import torch
        dtype = GRAM_F32 if src.dtype == torch.float32 else GRAM_BF16
        P = index.numel() if P is None else P
        self._ck(lib().gram_gather(self._h, _ptr(src), C.c_int64(src.shape[0]), _ptr(index), C.c_int64(P),
                                   C.c_int32(src.shape[1]), C.c_int(dtype), _ptr(E), _stream(stream)))

    def accumulate(self, dE, perm, seg_off, U, G, stream=None):
        self._ck(lib().gram_accumulate(self._h, _ptr(dE), _ptr(perm), _ptr(seg_off), C.c_int64(dE.shape[0]),
                                       C.c_int32(U), C.c_int32(dE.shape[1]), _ptr(G), _stream(stream)))

    def accumulate_multistep(self, dE, perm, seg_off, unique, U, n_items, table, touched_bits, stream=None):
        self._ck(lib().gram_accumulate_multistep(self._h, _ptr(dE), _ptr(perm), _ptr(seg_off), _ptr(unique),
                                                 C.c_int64(dE.shape[0]), C.c_int32(U), C.c_int32(dE.shape[1]),
                                                 C.c_int32(n_items), _ptr(table), _ptr(touched_bits), _stream(stream)))

    def touched_list(self, touched_bits, n_items, out_list, out_count, stream=None):
        self._ck(lib().gram_touched_list(self._h, _ptr(touched_bits), C.c_int32(n_items), _ptr(out_list),
                                         _ptr(out_count), _stream(stream)))

    def task(self, E, labels, B, dE, loss, stream=None):
        self._ck(lib().gram_task(self._h, _ptr(E), _ptr(labels), C.c_int32(B), _ptr(dE), _ptr(loss), _stream(stream)))

    def encoder_backward(self, G, items, U, stream=None):
        self._ck(lib().gram_encoder_backward(self._h, _ptr(G), _ptr(items), C.c_int32(U), _stream(stream)))

    def step(self, ids, labels, B, stream=None) -> GramStepReport:
        rep = GramStepReport()
        self._ck(lib().gram_step(self._h, _ptr(ids), _ptr(labels), C.c_int32(B), C.byref(rep), _stream(stream)))
        return rep

    def step_host(self, ids: np.ndarray, labels: np.ndarray, B, stream=None) -> GramStepReport:
        rep = GramStepReport()
        self._ck(lib().gram_step_host(self._h, _ptr(ids), _ptr(labels), C.c_int32(B), C.byref(rep), _stream(stream)))
        return rep

    def cache_fill(self, stream=None):
        self._ck(lib().gram_cache_fill(self._h, _stream(stream)))

    def window_reset(self, stream=None):
        self._ck(lib().gram_window_reset(self._h, _stream(stream)))

    def get_window(self, want_table=True, want_touched=True, want_cache=True):
        n, d = self.cfg.n_items, self.cfg.d
        table = np.empty((n, d), np.float32) if want_table else None
        touched = np.empty((n + 31) // 32, np.uint32) if want_touched else None
        cache = np.empty((n, d), np.float32) if want_cache else None
        self._ck(lib().gram_get_window(self._h, _ptr(table), _ptr(touched), _ptr(cache)))
        return table, touched, cache

    # checkpoint / resume
    def state_export(self):
        """(table, touched, cache, steps_in_window) of the open Multi-step window."""
        n, d = self.cfg.n_items, self.cfg.d
        table = np.empty((n, d), np.float32); touched = np.empty((n + 31) // 32, np.uint32); cache = np.empty((n, d), np.float32)
        steps = C.c_int32(0)
        self._ck(lib().gram_state_export(self._h, _ptr(table), _ptr(touched), _ptr(cache), C.byref(steps)))
        return table, touched, cache, steps.value

    def state_import(self, table, touched, cache, steps_in_window: int):
        table = None if table is None else np.ascontiguousarray(table, np.float32)
        touched = None if touched is None else np.ascontiguousarray(touched, np.uint32)
        cache = None if cache is None else np.ascontiguousarray(cache, np.float32)
        self._ck(lib().gram_state_import(self._h, _ptr(table), _ptr(touched), _ptr(cache), C.c_int32(int(steps_in_window))))

    def optimizer_export(self, module: int):
        """(m, v, updates) of one module; m and v are None for plain SGD."""
        n = self.param_count(module)
        adam = self.cfg.optimizer == GRAM_OPT_ADAM
        m = np.empty(n, np.float32) if adam else None
        v = np.empty(n, np.float32) if adam else None
        upd = C.c_int64(0)
        self._ck(lib().gram_optimizer_export(self._h, module, _ptr(m), _ptr(v), C.byref(upd)))
        return m, v, upd.value

    def optimizer_import(self, module: int, m, v, updates: int):
        m = None if m is None else np.ascontiguousarray(m, np.float32)
        v = None if v is None else np.ascontiguousarray(v, np.float32)
        self._ck(lib().gram_optimizer_import(self._h, module, _ptr(m), _ptr(v), C.c_int64(int(updates))))

    # measurement
    def profile(self, enable: bool):
        self._ck(lib().gram_profile(self._h, C.c_int(int(enable))))

    def profile_read(self) -> dict:
        """{kind: dict(ms, work, launches)} since the last profile() call."""
        out = {}
        for k, name in enumerate(KINDS):
            ms, work, n = C.c_double(0), C.c_double(0), C.c_int64(0)
            self._ck(lib().gram_profile_read(self._h, C.c_int(k), C.byref(ms), C.byref(work), C.byref(n)))
            out[name] = dict(ms=ms.value, work=work.value, launches=n.value)
        return out

    def profile_dump(self) -> dict:
        """{tag: dict(kind, ms, work, launches)} per call site since the last profile() call."""
        buf = C.create_string_buffer(16384)
        self._ck(lib().gram_profile_dump(self._h, buf, C.c_size_t(len(buf))))
        out = {}
        for line in buf.value.decode().splitlines():
            tag, kind, ms, work, n = line.split()
            out[tag] = dict(kind=KINDS[int(kind)], ms=float(ms), work=float(work), launches=int(n))
        return out

    def launch_count(self) -> int:
        n = C.c_int64(0)
        self._ck(lib().gram_launch_count(self._h, C.byref(n)))
        return n.value

    def gemm_bf16(self, A, a_kmajor, Bm, b_kmajor, Cm, bias, accumulate, M, N, K, stream=None):
        import torch
        self._ck(lib().gram_gemm_bf16(self._h, _ptr(A), C.c_int(int(a_kmajor)), _ptr(Bm), C.c_int(int(b_kmajor)),
                                      _ptr(Cm), C.c_int(int(Cm.dtype == torch.float32)), _ptr(bias),
                                      C.c_int(int(accumulate)), C.c_int64(M), C.c_int32(N), C.c_int64(K),
                                      _stream(stream)))


    def gemm_bf16_epilogue(self, A, a_kmajor, Bm, b_kmajor, Cm, M, N, K, bias=None, res=None, res_ln=None, gelu=False,
                           gelu_grad_out=None, gelu_grad_in=None, copy_bf16=None, accumulate=False, stream=None):
        """res_ln: (mean, rstd, gamma, beta) applied to `res` where it is read."""
        import torch
        e = GramGemmEpilogue()
        e.d_bias = _ptr(bias); e.d_res = _ptr(res)
        if res_ln is not None:
            e.d_res_mean, e.d_res_rstd, e.d_res_gamma, e.d_res_beta = (_ptr(t) for t in res_ln)
        e.d_gelu_grad_out = _ptr(gelu_grad_out); e.d_gelu_grad_in = _ptr(gelu_grad_in); e.d_copy_bf16 = _ptr(copy_bf16)
        e.gelu = int(gelu); e.accumulate = int(accumulate)
        self._ck(lib().gram_gemm_bf16_epilogue(self._h, _ptr(A), C.c_int(int(a_kmajor)), _ptr(Bm), C.c_int(int(b_kmajor)),
                                               _ptr(Cm), C.c_int(int(Cm.dtype == torch.float32)), C.byref(e), C.c_int64(M),
                                               C.c_int32(N), C.c_int64(K), _stream(stream)))


def accumulate_static(dE, perm, seg_off, U, G, stream=None, P=None, d=None):
    """gram_accumulate_static: the segmented sum with its scratch in a fixed array of the library, for
    callers that may not allocate device memory.  Needs no context.  Raises GramError with the
    library's message on failure."""
    err = C.create_string_buffer(256)
    P = dE.shape[0] if P is None else P
    d = dE.shape[1] if d is None else d
    st = lib().gram_accumulate_static(_ptr(dE), _ptr(perm), _ptr(seg_off), C.c_int64(P), C.c_int32(U), C.c_int32(d),
                                      _ptr(G), _stream(stream), err, C.c_size_t(len(err)))
    if st != 0:
        raise GramError(st, err.value.decode())
