"""ctypes binding over the C ABI of liblayerpipe.so (see include/layerpipe.h).

Argument marshalling only: every step of the training path runs in the library's
CUDA kernels.  torch is used for device memory (the workspace, the minibatch)
and streams.  Loading fails loudly if the library has not been built; there is
no fallback path.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblayerpipe.so")

LP_OK = 0
LP_ERR_INVALID_ARG, LP_ERR_UNSUPPORTED, LP_ERR_WORKSPACE = -1, -2, -3
LP_ERR_CUDA, LP_ERR_TIMEOUT, LP_ERR_NOT_READY = -4, -5, -6
LP_FC, LP_CONV = 0, 1
LP_ACT = {"none": 0, "relu": 1, "gelu": 2}
LP_SCHED_LAYERPIPE, LP_SCHED_FUSED_B = 0, 1
LP_F32, LP_BF16 = 0, 1
LP_CAPTURE_GRADS = 1
LP_TIME_TASKS = 2
LP_UNFUSED_UPDATE = 4
LP_SERIAL_TASKS = 8
LP_RECOMPUTE = 16
LP_TRACE_TASKS = 32


class lp_layer(C.Structure):
    _fields_ = [("kind", C.c_int), ("n_in", C.c_int), ("n_out", C.c_int), ("H", C.c_int), ("W", C.c_int),
                ("R", C.c_int), ("S", C.c_int), ("stride", C.c_int), ("pad", C.c_int), ("act", C.c_int),
                ("pool", C.c_int), ("has_bias", C.c_int)]


class lp_config(C.Structure):
    _fields_ = [("batch", C.c_int), ("lr", C.c_float), ("momentum", C.c_float), ("schedule", C.c_int),
                ("input_dtype", C.c_int), ("flags", C.c_uint)]


class LayerPipeError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("layerpipe error %d: %s" % (code, msg))
        self.code = code


_lib = None
_P = C.POINTER


def lib():
    """Load the shared library (once).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError("liblayerpipe.so is not built: run `python -m paper_2108_06629_b200.build` "
                          "(needs nvcc); there is no CPU fallback")
    L = C.CDLL(LIB_PATH)
    vp, ip, llp, fp = C.c_void_p, _P(C.c_int), _P(C.c_longlong), _P(C.c_float)
    sig = {
        "lp_plan": [_P(lp_layer), C.c_int, C.c_int, C.c_int, ip, ip, ip, llp, ip, llp, ip],
        "lp_plan_costs": [llp, llp, C.c_int, C.c_int, ip, ip, ip, llp, ip, llp, ip],
        "lp_workspace_size": [_P(lp_layer), C.c_int, C.c_int, ip, ip, _P(lp_config), _P(C.c_size_t)],
        "lp_create": [_P(vp), _P(lp_layer), C.c_int, C.c_int, ip, ip, _P(lp_config), _P(fp), _P(fp), vp, C.c_size_t],
        "lp_step": [vp, vp, vp, vp],
        "lp_flush": [vp, vp],
        "lp_get_weights": [vp, C.c_int, fp, fp, llp],
        "lp_get_grads": [vp, C.c_int, C.c_longlong, fp, fp],
        "lp_get_schedule": [vp, ip, ip, ip],
        "lp_debug_read": [vp, C.c_int, C.c_int, C.c_longlong, fp],
        "lp_debug_write": [vp, C.c_int, C.c_int, C.c_longlong, fp],
        "lp_debug_run_task": [vp, C.c_int, C.c_int, C.c_longlong],
        "lp_get_version_log": [vp, C.c_longlong, ip, ip, ip],
        "lp_get_loss": [vp, C.c_longlong, fp],
        "lp_device_status": [vp, ip],
        "lp_get_task_time": [vp, C.c_int, llp, _P(C.c_double)],
        "lp_reset_task_times": [vp],
        "lp_get_layer_task_time": [vp, C.c_int, C.c_int, llp, _P(C.c_double)],
        "lp_set_delta_split": [vp, ip, llp, ip],
        "lp_task_progress": [vp, C.c_char_p, C.c_int],
        "lp_get_task_timeline": [vp, C.c_int, C.c_int, _P(C.c_float), _P(C.c_float), _P(C.c_int)],
        "lp_set_tuning": [C.c_int, C.c_int, C.c_int],
        "lp_destroy": [vp],
        "lp_gemm_bf16": [C.c_int, C.c_int, C.c_int, C.c_int, vp, C.c_int, vp, C.c_int, vp, C.c_int, vp],
        "lp_softmax_xent_static": [vp, C.c_int, vp, vp, C.c_int, vp, C.c_int, C.c_int, vp],
        "lp_gemm_status": [ip],
        "lp_debug_gemm_starved": [C.c_int, C.c_int, C.c_int, vp, C.c_int, vp, C.c_int, vp, C.c_int, C.c_longlong, vp],
    }
    for name, args in sig.items():
        f = getattr(L, name)
        f.argtypes = args
        f.restype = C.c_int
    L.lp_kernel_launches.argtypes = [vp]
    L.lp_kernel_launches.restype = C.c_longlong
    L.lp_last_error.argtypes = [vp]
    L.lp_last_error.restype = C.c_char_p
    _lib = L
    return L


EXPORTS = ["lp_plan", "lp_plan_costs", "lp_workspace_size", "lp_create", "lp_step", "lp_flush",
           "lp_get_weights", "lp_get_grads", "lp_debug_read", "lp_debug_write", "lp_debug_run_task", "lp_get_schedule", "lp_get_version_log", "lp_get_loss",
           "lp_device_status", "lp_task_progress", "lp_get_task_time", "lp_reset_task_times", "lp_get_layer_task_time", "lp_set_delta_split", "lp_get_task_timeline", "lp_kernel_launches", "lp_set_tuning", "lp_last_error", "lp_destroy",
           "lp_gemm_bf16", "lp_gemm_status", "lp_debug_gemm_starved", "lp_softmax_xent_static"]


def _check(rc, h=None):
    if rc != LP_OK:
        raise LayerPipeError(rc, (lib().lp_last_error(h) or b"").decode())


def _layers_array(layers):
    arr = (lp_layer * len(layers))()
    for i, l in enumerate(layers):
        arr[i].kind = LP_FC if l["kind"] == "fc" else LP_CONV
        arr[i].n_in, arr[i].n_out = l["n_in"], l["n_out"]
        arr[i].H, arr[i].W = l.get("H", 0), l.get("W", 0)
        arr[i].R, arr[i].S = l.get("R", 0), l.get("S", 0)
        arr[i].stride, arr[i].pad = l.get("stride", 0), l.get("pad", 0)
        arr[i].act = LP_ACT[l["act"]]
        arr[i].pool = l.get("pool", 0)
        arr[i].has_bias = 1 if l.get("bias", True) else 0
    return arr


def _int_array(xs):
    return None if xs is None else (C.c_int * len(xs))(*[int(x) for x in xs])


def lp_plan(layers, batch, n_stages):
    """Algorithm 1 on the integer MAC model.  Returns a dict like the oracle's."""
    n = len(layers)
    st, dl, ps = (C.c_int * n)(), (C.c_int * n)(), (C.c_int * (2 * n))()
    pa = (C.c_longlong * (2 * n))()
    used, rounds, Tp = C.c_int(), C.c_int(), C.c_longlong()
    _check(lib().lp_plan(_layers_array(layers), n, batch, n_stages, st, dl, ps, pa, C.byref(used), C.byref(Tp),
                         C.byref(rounds)))
    return dict(stage=list(st), delay=list(dl), piece_stage=list(ps), piece_amount=list(pa), used=used.value,
                T_p=Tp.value, relax_rounds=rounds.value)


def lp_plan_costs(T_fix, T_flex, n_stages):
    n = len(T_fix)
    st, dl, ps = (C.c_int * n)(), (C.c_int * n)(), (C.c_int * (2 * n))()
    pa = (C.c_longlong * (2 * n))()
    used, rounds, Tp = C.c_int(), C.c_int(), C.c_longlong()
    fx = (C.c_longlong * n)(*[int(x) for x in T_fix])
    fl = (C.c_longlong * n)(*[int(x) for x in T_flex])
    _check(lib().lp_plan_costs(fx, fl, n, n_stages, st, dl, ps, pa, C.byref(used), C.byref(Tp), C.byref(rounds)))
    return dict(stage=list(st), delay=list(dl), piece_stage=list(ps), piece_amount=list(pa), used=used.value,
                T_p=Tp.value, relax_rounds=rounds.value)


def _config(batch, lr, momentum, schedule, input_dtype, flags):
    return lp_config(batch, lr, momentum, schedule, input_dtype, flags)


def lp_workspace_size(layers, n_stages, stage, delays, batch, lr=0.01, momentum=0.0,
                      schedule=LP_SCHED_LAYERPIPE, input_dtype=LP_F32, flags=0):
    out = C.c_size_t()
    cfg = _config(batch, lr, momentum, schedule, input_dtype, flags)
    _check(lib().lp_workspace_size(_layers_array(layers), len(layers), n_stages, _int_array(stage),
                                   _int_array(delays), C.byref(cfg), C.byref(out)))
    return out.value


def lp_set_tuning(tile_n=0, stages=0, split_k=0):
    _check(lib().lp_set_tuning(tile_n, stages, split_k))


class Trainer:
    """lp_create / lp_step / lp_flush / lp_get_* on one handle.  The workspace is a
    torch uint8 tensor owned by this object."""

    def __init__(self, layers, batch, n_stages, delays=None, stage=None, lr=0.01, momentum=0.0,
                 schedule=LP_SCHED_LAYERPIPE, input_dtype=LP_F32, flags=0, W0=None, b0=None, device="cuda:0"):
        import torch
        self.torch = torch
        self.layers = layers
        self.batch = batch
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        L = lib()
        n = len(layers)
        arr = _layers_array(layers)
        cfg = _config(batch, lr, momentum, schedule, input_dtype, flags)
        size = C.c_size_t()
        _check(L.lp_workspace_size(arr, n, n_stages, _int_array(stage), _int_array(delays), C.byref(cfg),
                                   C.byref(size)))
        self.workspace_bytes = size.value
        self.workspace = torch.empty(size.value + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        Wp = (_P(C.c_float) * n)()
        bp = (_P(C.c_float) * n)()
        self._keep = []
        for i in range(n):
            w = np.ascontiguousarray(W0[i], dtype=np.float32)
            self._keep.append(w)
            Wp[i] = w.ctypes.data_as(_P(C.c_float))
            if b0 is not None and b0[i] is not None:
                b = np.ascontiguousarray(b0[i], dtype=np.float32)
                self._keep.append(b)
                bp[i] = b.ctypes.data_as(_P(C.c_float))
        h = C.c_void_p()
        _check(L.lp_create(C.byref(h), arr, n, n_stages, _int_array(stage), _int_array(delays), C.byref(cfg), Wp, bp,
                           C.c_void_p(base), size.value))
        self.h = h
        self._keep = []

    # ---- the calls ---------------------------------------------------------
    def step(self, batch_dev, labels_dev, stream=None):
        s = self.torch.cuda.current_stream(self.device).cuda_stream if stream is None else stream
        _check(lib().lp_step(self.h, C.c_void_p(batch_dev.data_ptr()), C.c_void_p(labels_dev.data_ptr()),
                             C.c_void_p(s)), self.h)

    def flush(self, stream=None):
        s = self.torch.cuda.current_stream(self.device).cuda_stream if stream is None else stream
        _check(lib().lp_flush(self.h, C.c_void_p(s)), self.h)

    def get_weights(self, layer):
        l = self.layers[layer]
        shape = (l["n_out"], l["n_in"]) if l["kind"] == "fc" else (l["n_out"], l["R"], l["S"], l["n_in"])
        W = np.empty(shape, dtype=np.float32)
        b = np.empty(l["n_out"], dtype=np.float32)
        ver = C.c_longlong()
        _check(lib().lp_get_weights(self.h, layer, W.ctypes.data_as(_P(C.c_float)),
                                    b.ctypes.data_as(_P(C.c_float)), C.byref(ver)), self.h)
        return W, b, ver.value

    def get_grads(self, layer, step):
        l = self.layers[layer]
        shape = (l["n_out"], l["n_in"]) if l["kind"] == "fc" else (l["n_out"], l["R"], l["S"], l["n_in"])
        dW = np.empty(shape, dtype=np.float32)
        db = np.empty(l["n_out"], dtype=np.float32)
        _check(lib().lp_get_grads(self.h, layer, step, dW.ctypes.data_as(_P(C.c_float)),
                                  db.ctypes.data_as(_P(C.c_float))), self.h)
        return dW, db

    # ---- verification access (see the header: lp_debug_*) -------------------
    BUF = {"input": 0, "z": 1, "delta": 2, "logits": 3, "labels": 4, "loss": 5, "ring_w": 6, "ring_b": 7,
           "master_w": 8, "master_b": 9, "mom_w": 10, "mom_b": 11, "grad_w": 12, "grad_b": 13, "pool_idx": 14}
    TASK = {"forward": 0, "loss": 1, "delta": 2, "G": 3, "update": 4}

    def _buf_shape(self, buf, layer):
        l = self.layers[layer]
        classes = self.layers[-1]["n_out"]
        B = self.batch
        if l["kind"] == "conv":
            H, W = l["H"], l["W"]
            Ho = (H + 2 * l["pad"] - l["R"]) // l["stride"] + 1          # delta^l lives on the layer's output grid
            Wo = (W + 2 * l["pad"] - l["S"]) // l["stride"] + 1
            Hp, Wp = (Ho // 2, Wo // 2) if l.get("pool", 0) else (Ho, Wo)
            wshape = (l["n_out"], l["R"], l["S"], l["n_in"])
            shapes = {"input": (B, H, W, l["n_in"]), "delta": (B, Ho, Wo, l["n_out"]),
                      "pool_idx": (B, Hp, Wp, l["n_out"])}
        else:
            wshape = (l["n_out"], l["n_in"])
            shapes = {"input": (B, l["n_in"]), "z": (B, l["n_out"]), "delta": (B, l["n_out"])}
        shapes.update({"logits": (B, classes), "labels": (B,), "loss": (1,), "ring_w": wshape, "master_w": wshape,
                       "mom_w": wshape, "grad_w": wshape})
        return shapes.get(buf, (l["n_out"],))

    def debug_read(self, buf, layer, index):
        out = np.empty(self._buf_shape(buf, layer), dtype=np.float32)
        _check(lib().lp_debug_read(self.h, self.BUF[buf], layer, index, out.ctypes.data_as(_P(C.c_float))), self.h)
        return out

    def debug_write(self, buf, layer, index, value):
        v = np.ascontiguousarray(np.asarray(value, dtype=np.float32).reshape(self._buf_shape(buf, layer)))
        _check(lib().lp_debug_write(self.h, self.BUF[buf], layer, index, v.ctypes.data_as(_P(C.c_float))), self.h)

    def debug_run_task(self, task, layer, step):
        _check(lib().lp_debug_run_task(self.h, self.TASK[task], layer, step), self.h)

    def get_schedule(self):
        n = len(self.layers)
        a, b, c = (C.c_int * n)(), (C.c_int * n)(), (C.c_int * n)()
        _check(lib().lp_get_schedule(self.h, a, b, c), self.h)
        return list(a), list(b), list(c)

    def get_version_log(self, step):
        n = len(self.layers)
        a, b, c = (C.c_int * n)(), (C.c_int * n)(), (C.c_int * n)()
        _check(lib().lp_get_version_log(self.h, step, a, b, c), self.h)
        return list(a), list(b), list(c)

    def get_loss(self, step):
        v = C.c_float()
        _check(lib().lp_get_loss(self.h, step, C.byref(v)), self.h)
        return v.value

    def device_status(self):
        d = C.c_int()
        rc = lib().lp_device_status(self.h, C.byref(d))
        return rc, d.value

    def task_time(self, task):
        """(launches, total milliseconds) of one task kind; needs flags=LP_TIME_TASKS."""
        k = dict(self.TASK, cast=5)[task]
        n, ms = C.c_longlong(), C.c_double()
        _check(lib().lp_get_task_time(self.h, k, C.byref(n), C.byref(ms)), self.h)
        return n.value, ms.value

    def task_timeline(self, task, capacity=4096):
        """(start_ms, end_ms) arrays of the timed launches of one task kind, in launch order,
        relative to the first event timed since the last reset; needs flags=LP_TIME_TASKS."""
        k = dict(self.TASK, cast=5)[task]
        st = np.zeros(capacity, dtype=np.float32)
        en = np.zeros(capacity, dtype=np.float32)
        n = C.c_int()
        _check(lib().lp_get_task_timeline(self.h, k, capacity, st.ctypes.data_as(_P(C.c_float)),
                                          en.ctypes.data_as(_P(C.c_float)), C.byref(n)), self.h)
        return st[:n.value], en[:n.value]

    def layer_task_time(self, task, layer):
        """(launches, total milliseconds) of one task kind of one layer; needs flags=LP_TIME_TASKS."""
        k = dict(self.TASK, cast=5)[task]
        n, ms = C.c_longlong(), C.c_double()
        _check(lib().lp_get_layer_task_time(self.h, k, layer, C.byref(n), C.byref(ms)), self.h)
        return n.value, ms.value

    def task_progress(self):
        """Text: unfinished tasks per scheduler stream and the status word (flags=LP_TRACE_TASKS).
        Does not wait for the device; callable from a second thread."""
        buf = C.create_string_buffer(4096)
        _check(lib().lp_task_progress(self.h, buf, 4096), self.h)
        return buf.value.decode()

    def set_delta_split(self, piece_stage, piece_amount):
        """Divide the delta contractions by output columns as a plan's pieces say (before the first
        step).  Returns the first column of delta' per layer (0 = unsplit)."""
        n = len(self.layers)
        ps = (C.c_int * (2 * n))(*[int(x) for x in piece_stage])
        pa = (C.c_longlong * (2 * n))(*[int(x) for x in piece_amount])
        out = (C.c_int * n)()
        _check(lib().lp_set_delta_split(self.h, ps, pa, out), self.h)
        return list(out)

    def reset_task_times(self):
        _check(lib().lp_reset_task_times(self.h), self.h)

    def kernel_launches(self):
        return lib().lp_kernel_launches(self.h)

    def close(self):
        if getattr(self, "h", None):
            lib().lp_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def lp_gemm_bf16(which, M, N, K, A, lda, B, ldb, Cout, ldc, stream=None):
    """A, B: torch bf16 device tensors; Cout: torch fp32 device tensor."""
    import torch
    s = torch.cuda.current_stream().cuda_stream if stream is None else stream
    _check(lib().lp_gemm_bf16(which, M, N, K, C.c_void_p(A.data_ptr()), lda, C.c_void_p(B.data_ptr()), ldb,
                              C.c_void_p(Cout.data_ptr()), ldc, C.c_void_p(s)))


def lp_gemm_status():
    """(return code, status word) of the lp_gemm_bf16 launches since the last call; clears the word."""
    d = C.c_int()
    rc = lib().lp_gemm_status(C.byref(d))
    return rc, d.value


def lp_debug_gemm_starved(M, N, K, A, lda, B, ldb, Cout, ldc, limit_cycles, stream=None):
    """Forward contraction whose producer skips the last k-block: a bounded wait must run out."""
    import torch
    s = torch.cuda.current_stream().cuda_stream if stream is None else stream
    _check(lib().lp_debug_gemm_starved(M, N, K, C.c_void_p(A.data_ptr()), lda, C.c_void_p(B.data_ptr()), ldb,
                                       C.c_void_p(Cout.data_ptr()), ldc, limit_cycles, C.c_void_p(s)))


LP_XENT_STATIC_MAX_BATCH = 16384


def lp_softmax_xent_static(logits, labels, delta, loss, classes, stream=None):
    """Loss kernel on caller-owned torch tensors, no handle and no allocation inside the
    library: logits fp32 [batch][ld], labels int32 [batch], delta bf16 [batch][ld_delta]
    (output), loss fp32 [1] (output).  Returns the library's status code."""
    import torch
    s = torch.cuda.current_stream().cuda_stream if stream is None else stream
    return lib().lp_softmax_xent_static(C.c_void_p(logits.data_ptr()), logits.stride(0),
                                        C.c_void_p(labels.data_ptr()), C.c_void_p(delta.data_ptr()),
                                        delta.stride(0), C.c_void_p(loss.data_ptr()), logits.shape[0], classes,
                                        C.c_void_p(s))
