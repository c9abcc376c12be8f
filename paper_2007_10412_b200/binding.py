"""ctypes binding of librad_b200.so: argument marshalling only.

Every function here has the name of the C entry point it calls (include/rad.h)
and passes torch tensors by data pointer plus the current CUDA stream.  torch
is used for device memory and streams; no arithmetic of the method happens in
Python.  There is no CPU fallback: a missing library or a negative return code
raises.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librad_b200.so")

RAD_F32, RAD_BF16 = 0, 1
RAD_DIFFERENT_SAMPLE, RAD_SAME_SAMPLE, RAD_PROJECT, RAD_ROWS_SAMPLE, RAD_REDRAWN_SAMPLE = 0, 1, 2, 3, 4
RAD_ACT_NONE, RAD_ACT_RELU, RAD_ACT_GELU = 0, 1, 2
RAD_DEV_ECAPACITY, RAD_DEV_ETIMEOUT = 1, 2
TILE_ROWS, TILE_COLS, VALUE_ALIGN = 64, 128, 8

DTYPES = {"f32": RAD_F32, "bf16": RAD_BF16, torch.float32: RAD_F32, torch.bfloat16: RAD_BF16}
VARIANTS = {"different": RAD_DIFFERENT_SAMPLE, "same": RAD_SAME_SAMPLE, "project": RAD_PROJECT, "rows": RAD_ROWS_SAMPLE,
            "redrawn": RAD_REDRAWN_SAMPLE}
LAWS = {"bernoulli": 0, "replace": 1, "fixed": 2}
ACTS = {"none": RAD_ACT_NONE, "relu": RAD_ACT_RELU, "gelu": RAD_ACT_GELU}
TORCH_DTYPE = {RAD_F32: torch.float32, RAD_BF16: torch.bfloat16}


class RadError(RuntimeError):
    pass


class rad_store(C.Structure):
    _fields_ = [("variant", C.c_int32), ("dtype", C.c_int32), ("B", C.c_int64), ("D", C.c_int64),
                ("p", C.c_float), ("layer", C.c_uint32), ("step", C.c_uint32), ("seed", C.c_uint64),
                ("values", C.c_void_p), ("values_capacity", C.c_int64), ("values_ld", C.c_int64),
                ("keepbits", C.c_void_p), ("offsets", C.c_void_p), ("nnz", C.c_void_p),
                ("relubits", C.c_void_p), ("law", C.c_int32)]


class rad_store_sizes(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("values_worst", "values_typical", "values_ld_worst",
                                         "values_ld_typical", "keepbits_words", "offsets_words",
                                         "relubits_words", "workspace_bytes")]


class rad_mlp_desc(C.Structure):
    _fields_ = [("L", C.c_int32), ("act", C.c_int32), ("dtype", C.c_int32), ("variant", C.c_int32),
                ("dims", C.POINTER(C.c_int64)), ("B", C.c_int64), ("p", C.c_float), ("step", C.c_uint32),
                ("seed", C.c_uint64), ("law", C.c_int32)]


class rad_irnn_desc(C.Structure):
    _fields_ = [("B", C.c_int64), ("T", C.c_int64), ("Hd", C.c_int64), ("C", C.c_int64), ("variant", C.c_int32),
                ("p", C.c_float), ("seed", C.c_uint64), ("step0", C.c_uint32)]


class rad_cnn_desc(C.Structure):
    _fields_ = [("B", C.c_int64), ("H", C.c_int64), ("W", C.c_int64), ("Cin", C.c_int64), ("n_conv", C.c_int32),
                ("n_fc", C.c_int32), ("conv_channels", C.POINTER(C.c_int64)), ("fc_dims", C.POINTER(C.c_int64)),
                ("dtype", C.c_int32), ("variant", C.c_int32), ("p", C.c_float), ("step", C.c_uint32),
                ("seed", C.c_uint64)]


class rad_step_stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("value_bytes", "index_bytes", "relu_bytes", "preact_bytes",
                                         "unsampled_bytes", "full_backprop_bytes")]


EXPORTS = ["rad_keep_threshold", "rad_effective_p", "rad_scale", "rad_store_size_query", "rad_set_store_kernel",
           "rad_draws_per_row", "rad_replace_scale", "rad_store_size_query_law", "rad_rademacher",
           "rad_linear_forward_store", "rad_linear_forward_store_static", "rad_weight_grad_workspace", "rad_linear_weight_grad",
           "rad_linear_forward", "rad_store_index", "rad_linear_forward_fill", "rad_softmax_xent", "rad_input_grad_workspace", "rad_linear_input_grad",
           "rad_mlp_workspace", "rad_mlp_held_bytes", "rad_mlp_step", "rad_irnn_workspace", "rad_irnn_step", "rad_cnn_workspace", "rad_cnn_step", "rad_launch_count", "rad_sm_pairs", "rad_strerror", "rad_version",
           "rad_set_wait_limit_ns", "rad_wait_probe", "rad_set_conv_kernel"]

_lib = None


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RadError(f"{LIB_PATH} is missing: run `python -m paper_2007_10412_b200.build`")
        L = C.CDLL(LIB_PATH)
        L.rad_keep_threshold.restype = C.c_uint32
        L.rad_keep_threshold.argtypes = [C.c_float]
        L.rad_effective_p.restype = C.c_float
        L.rad_effective_p.argtypes = [C.c_float]
        L.rad_scale.restype = C.c_float
        L.rad_scale.argtypes = [C.c_float]
        L.rad_strerror.restype = C.c_char_p
        L.rad_strerror.argtypes = [C.c_int]
        L.rad_version.restype = C.c_char_p
        L.rad_launch_count.restype = C.c_int64
        i32, i64, f32, vp = C.c_int32, C.c_int64, C.c_float, C.c_void_p
        L.rad_set_store_kernel.argtypes = [i32]
        L.rad_set_conv_kernel.argtypes = [i32]
        L.rad_draws_per_row.restype = i64
        L.rad_draws_per_row.argtypes = [f32, i64]
        L.rad_replace_scale.restype = f32
        L.rad_replace_scale.argtypes = [f32, i64]
        L.rad_rademacher.argtypes = [i32, i64, f32, i64, C.c_uint64, C.c_uint32, C.c_uint32, vp, vp]
        L.rad_store_size_query_law.argtypes = [i32, i32, i32, i64, i64, f32, C.POINTER(rad_store_sizes)]
        L.rad_store_size_query.argtypes = [i32, i32, i64, i64, f32, C.POINTER(rad_store_sizes)]
        L.rad_linear_forward_store.argtypes = [vp, i64, C.POINTER(rad_store), vp, i64, vp, vp]
        L.rad_linear_forward_store_static.argtypes = [vp, i64, C.POINTER(rad_store), vp, vp]
        L.rad_weight_grad_workspace.argtypes = [C.POINTER(rad_store), i64, C.POINTER(i64)]
        L.rad_linear_weight_grad.argtypes = [C.POINTER(rad_store), vp, i64, i64, vp, i64, vp, i64, vp, vp]
        L.rad_linear_forward.argtypes = [i32, i32, i64, i64, i64, vp, i64, vp, i64, vp, vp, i64, vp, i64,
                                         vp, i64, vp, vp, vp]
        L.rad_store_index.argtypes = [C.POINTER(rad_store), vp, vp]
        L.rad_set_wait_limit_ns.restype = C.c_uint64
        L.rad_set_wait_limit_ns.argtypes = [C.c_uint64]
        L.rad_wait_probe.argtypes = [i32, C.c_uint64, vp, vp]
        L.rad_linear_forward_fill.argtypes = [i32, i32, i64, i64, i64, vp, i64, vp, i64, vp, vp, i64, vp, i64, vp,
                                              C.POINTER(rad_store), i32, vp, i64, vp, vp]
        L.rad_softmax_xent.argtypes = [i32, i64, i64, vp, i64, vp, vp, vp, i64, vp, i64, vp]
        L.rad_input_grad_workspace.argtypes = [i64, i64, C.POINTER(i64)]
        L.rad_linear_input_grad.argtypes = [i32, i64, i64, i64, vp, i64, vp, i64, vp, vp, i64, vp, i64, vp,
                                            vp, i64, vp, vp]
        L.rad_mlp_workspace.argtypes = [C.POINTER(rad_mlp_desc), C.POINTER(i64), C.POINTER(rad_step_stats)]
        L.rad_mlp_held_bytes.argtypes = [C.POINTER(rad_mlp_desc), C.POINTER(i64), C.POINTER(rad_step_stats)]
        L.rad_irnn_workspace.argtypes = [C.POINTER(rad_irnn_desc), C.POINTER(i64), C.POINTER(rad_step_stats)]
        L.rad_irnn_step.argtypes = [C.POINTER(rad_irnn_desc)] + [vp] * 15 + [vp, i64, vp, vp]
        L.rad_cnn_workspace.argtypes = [C.POINTER(rad_cnn_desc), C.POINTER(i64), C.POINTER(rad_step_stats)]
        L.rad_cnn_step.argtypes = [C.POINTER(rad_cnn_desc), vp, vp] + [C.POINTER(vp)] * 8 + [vp, vp, vp, i64, vp, vp]
        L.rad_mlp_step.argtypes = [C.POINTER(rad_mlp_desc), vp, vp, C.POINTER(vp), C.POINTER(vp),
                                   C.POINTER(vp), C.POINTER(vp), vp, vp, vp, i64, vp, vp]
        for name in EXPORTS:
            fn = getattr(L, name)
            if fn.restype is C.c_int:
                fn.restype = C.c_int
        _lib = L
    return _lib


def _check(rc, what):
    if rc != 0:
        raise RadError(f"{what} failed: {lib().rad_strerror(rc).decode()} ({rc})")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ld(t):
    return 0 if t is None else t.stride(0)


def rad_keep_threshold(p):
    return int(lib().rad_keep_threshold(p))


def rad_effective_p(p):
    return float(lib().rad_effective_p(p))


def rad_scale(p):
    return float(lib().rad_scale(p))


def rad_launch_count():
    return int(lib().rad_launch_count())


def rad_sm_pairs():
    """SM pairs the tensor-core kernels keep resident on the current device (74 where there is none to ask)."""
    return int(lib().rad_sm_pairs())


def rad_version():
    return lib().rad_version().decode()


def rad_store_size_query(variant, dtype, B, D, p):
    out = rad_store_sizes()
    _check(lib().rad_store_size_query(VARIANTS[variant], DTYPES[dtype], B, D, p, C.byref(out)),
           "rad_store_size_query")
    return out


def rad_store_size_query_law(variant, dtype, law, B, D, p):
    out = rad_store_sizes()
    _check(lib().rad_store_size_query_law(VARIANTS[variant], DTYPES[dtype], LAWS[law], B, D, p, C.byref(out)),
           "rad_store_size_query_law")
    return out


def rad_rademacher(dtype, D, fraction, ld, seed, layer, step, out):
    """Writes the D x ld sign matrix of the projection variant to `out` (columns beyond k are zero)."""
    _check(lib().rad_rademacher(DTYPES[dtype], D, fraction, ld, seed, layer, step, _ptr(out), _stream()),
           "rad_rademacher")


def rad_draws_per_row(fraction, D):
    return int(lib().rad_draws_per_row(fraction, D))


def rad_replace_scale(fraction, D):
    return float(lib().rad_replace_scale(fraction, D))


class Store:
    """Device buffers of one layer's compact store plus the host struct that describes them."""

    def __init__(self, variant, dtype, B, D, p, seed=0, layer=0, step=0, relu_bits=True, capacity="typical",
                 device="cuda", law="bernoulli"):
        self.variant, self.dtype, self.B, self.D, self.p, self.law = variant, dtype, B, D, p, law
        sz = rad_store_size_query_law(variant, dtype, law, B, D, p)
        self.sizes = sz
        cap = {"typical": sz.values_typical, "worst": sz.values_worst}.get(capacity, capacity)
        ld = 0
        if variant in ("same", "project", "rows"):
            ld = {"typical": sz.values_ld_typical, "worst": sz.values_ld_worst}.get(capacity, capacity)
            cap = B * ld
        tdt = TORCH_DTYPE[DTYPES[dtype]]
        self.values = torch.empty(max(int(cap), 8), dtype=tdt, device=device)
        self.keepbits = torch.empty(sz.keepbits_words, dtype=torch.int32, device=device)
        self.offsets = torch.empty(max(sz.offsets_words, 1), dtype=torch.int32, device=device)
        self.nnz = torch.zeros(2, dtype=torch.int64, device=device)
        self.relubits = torch.empty(sz.relubits_words, dtype=torch.int32, device=device) if relu_bits else None
        self.workspace = torch.empty(sz.workspace_bytes, dtype=torch.uint8, device=device)
        self.c = rad_store(VARIANTS[variant], DTYPES[dtype], B, D, p, layer, step, seed,
                           self.values.data_ptr(), int(cap), int(ld),
                           self.keepbits.data_ptr() if sz.keepbits_words > 0 else None,
                           self.offsets.data_ptr(), self.nnz.data_ptr(),
                           self.relubits.data_ptr() if relu_bits else None, LAWS[law])

    def held_bytes(self):
        """Bytes this store holds between forward and backward (values as reserved, indices, ReLU bits)."""
        es = self.values.element_size()
        return dict(value_bytes=int(self.c.values_capacity) * es,
                    index_bytes=(self.keepbits.numel() + self.offsets.numel()) * 4,
                    relu_bytes=0 if self.relubits is None else self.relubits.numel() * 4)


def rad_linear_forward_store(A, store, dev_status=None):
    _check(lib().rad_linear_forward_store(_ptr(A), A.stride(0), C.byref(store.c), _ptr(store.workspace),
                                          store.workspace.numel(), _ptr(dev_status), _stream()),
           "rad_linear_forward_store")


STORE_KERNELS = {"auto": 0, "generic": 1, "pipelined": 2}


def rad_set_store_kernel(which):
    """Selects the different-sample store kernel ("auto", "generic", "pipelined"); returns the previous name."""
    prev = lib().rad_set_store_kernel(STORE_KERNELS[which])
    if prev < 0:
        _check(prev, "rad_set_store_kernel")
    return {v: k for k, v in STORE_KERNELS.items()}[prev]


CONV_KERNELS = {"auto": 0, "simt": 1, "tensor": 2}


def rad_set_conv_kernel(which):
    """Selects the kernels of the 3x3 convolutions ("auto", "simt", "tensor"); returns the previous name."""
    prev = lib().rad_set_conv_kernel(CONV_KERNELS[which])
    if prev < 0:
        _check(prev, "rad_set_conv_kernel")
    return {v: k for k, v in CONV_KERNELS.items()}[prev]


STATIC_STORE_MAX_TILES = 131072


def rad_linear_forward_store_static(A, store, dev_status=None):
    """The different-sample store for callers that may not allocate device memory while running.

    Same inputs and outputs as rad_linear_forward_store, but the kernel's scratch comes from a
    fixed array inside the library (at most STATIC_STORE_MAX_TILES tiles of 64 x 128), so nothing
    is allocated by the call; `store.workspace` is not used.  Calls on one device share that array:
    issue them on one stream, or otherwise ordered, never concurrently.
    """
    _check(lib().rad_linear_forward_store_static(_ptr(A), A.stride(0), C.byref(store.c), _ptr(dev_status),
                                                 _stream()), "rad_linear_forward_store_static")


def rad_weight_grad_workspace(store, H):
    out = C.c_int64(0)
    _check(lib().rad_weight_grad_workspace(C.byref(store.c), H, C.byref(out)), "rad_weight_grad_workspace")
    return out.value


def rad_linear_weight_grad(store, dZ, dW, workspace=None, dev_status=None):
    H = dZ.shape[1]
    if workspace is None:
        workspace = torch.empty(max(rad_weight_grad_workspace(store, H), 256), dtype=torch.uint8, device=dZ.device)
    _check(lib().rad_linear_weight_grad(C.byref(store.c), _ptr(dZ), dZ.stride(0), H, _ptr(dW), dW.stride(0),
                                        _ptr(workspace), workspace.numel(), _ptr(dev_status), _stream()),
           "rad_linear_weight_grad")
    return dW


def rad_linear_forward(A, W, bias, act, out_act=None, out_z=None, out_zlow=None, relubits=None, dev_status=None):
    B, D = A.shape
    H = W.shape[1]
    _check(lib().rad_linear_forward(DTYPES[A.dtype], ACTS[act], B, D, H, _ptr(A), A.stride(0), _ptr(W),
                                    W.stride(0), _ptr(bias), _ptr(out_act), _ld(out_act), _ptr(out_z),
                                    _ld(out_z), _ptr(out_zlow), _ld(out_zlow), _ptr(relubits),
                                    _ptr(dev_status), _stream()), "rad_linear_forward")


WAIT_PROBES = {"pair_barrier": 0, "pipe_barrier": 1, "lookback": 2}


def rad_set_wait_limit_ns(limit_ns):
    """Sets the time after which device-side waits give up (0 only reads); returns the previous value."""
    return int(lib().rad_set_wait_limit_ns(limit_ns))


def rad_wait_probe(which, limit_ns, dev_status):
    """Lets one of the kernels' bounded waits run out on purpose (a tiny kernel; nothing faults or hangs)."""
    _check(lib().rad_wait_probe(WAIT_PROBES[which], limit_ns, _ptr(dev_status), _stream()), "rad_wait_probe")


def rad_store_index(store, dev_status=None):
    """Keep bits, row offsets, tile offsets and nnz of a different-sample store from its key alone."""
    _check(lib().rad_store_index(C.byref(store.c), _ptr(dev_status), _stream()), "rad_store_index")


def rad_linear_forward_fill(A, W, bias, act, out_act, next_store, out_zlow=None, relubits=None, index_ready=False,
                            dev_status=None):
    """Forward of a hidden layer whose epilogue also fills `next_store` from the activations it holds."""
    B, D = A.shape
    H = W.shape[1]
    ws = next_store.workspace
    _check(lib().rad_linear_forward_fill(DTYPES[A.dtype], ACTS[act], B, D, H, _ptr(A), A.stride(0), _ptr(W),
                                         W.stride(0), _ptr(bias), _ptr(out_act), _ld(out_act), _ptr(out_zlow),
                                         _ld(out_zlow), _ptr(relubits), C.byref(next_store.c),
                                         1 if index_ready else 0, _ptr(ws), 0 if ws is None else ws.numel(),
                                         _ptr(dev_status), _stream()), "rad_linear_forward_fill")


def rad_softmax_xent(logits, labels, loss, dZ, workspace=None):
    B, Cn = logits.shape
    if workspace is None:
        workspace = torch.empty(B * 4, dtype=torch.uint8, device=logits.device)
    _check(lib().rad_softmax_xent(DTYPES[dZ.dtype], B, Cn, _ptr(logits), logits.stride(0), _ptr(labels),
                                  _ptr(loss), _ptr(dZ), dZ.stride(0), _ptr(workspace), workspace.numel(),
                                  _stream()), "rad_softmax_xent")


def rad_input_grad_workspace(B, H):
    out = C.c_int64(0)
    _check(lib().rad_input_grad_workspace(B, H, C.byref(out)), "rad_input_grad_workspace")
    return out.value


def rad_linear_input_grad(dZ, W, relubits_prev=None, z_prev=None, dZ_prev=None, db=None, workspace=None,
                          dev_status=None):
    B, H = dZ.shape
    D = W.shape[0]
    if workspace is None:
        workspace = torch.empty(rad_input_grad_workspace(B, H), dtype=torch.uint8, device=dZ.device)
    _check(lib().rad_linear_input_grad(DTYPES[dZ.dtype], B, D, H, _ptr(dZ), dZ.stride(0), _ptr(W), W.stride(0),
                                       _ptr(relubits_prev), _ptr(z_prev), _ld(z_prev), _ptr(dZ_prev),
                                       _ld(dZ_prev), _ptr(db), _ptr(workspace), workspace.numel(),
                                       _ptr(dev_status), _stream()), "rad_linear_input_grad")


def rad_mlp_workspace(dims, B, dtype="f32", act="relu", variant="different", p=0.1, law="bernoulli"):
    """(workspace bytes, rad_step_stats) of a net shape; allocates nothing."""
    dims_c = (C.c_int64 * len(dims))(*dims)
    desc = rad_mlp_desc(len(dims) - 1, ACTS[act], DTYPES[dtype], VARIANTS[variant], dims_c, B, p, 0, 0, LAWS[law])
    nbytes, stats = C.c_int64(0), rad_step_stats()
    _check(lib().rad_mlp_workspace(C.byref(desc), C.byref(nbytes), C.byref(stats)), "rad_mlp_workspace")
    return nbytes.value, stats


def rad_mlp_held_bytes(net, nnz_host):
    """rad_step_stats of the step that left `nnz_host` (the 2 L counts of MLPStep.nnz, copied to the host).
    `net`: an MLPStep, or the tuple (dims, B, dtype, act, variant, p, law) of a net shape."""
    if isinstance(net, tuple):
        dims, B, dtype, act, variant, p, law = net
        dims_c = (C.c_int64 * len(dims))(*dims)
        desc = rad_mlp_desc(len(dims) - 1, ACTS[act], DTYPES[dtype], VARIANTS[variant], dims_c, B, p, 0, 0, LAWS[law])
    else:
        desc = net.desc
    arr = (C.c_int64 * len(nnz_host))(*[int(v) for v in nnz_host])
    stats = rad_step_stats()
    _check(lib().rad_mlp_held_bytes(C.byref(desc), arr, C.byref(stats)), "rad_mlp_held_bytes")
    return stats


class MLPStep:
    """Owns the workspace and pointer tables of rad_mlp_step for one net shape."""

    def __init__(self, dims, B, dtype="f32", act="relu", variant="different", p=0.1, device="cuda",
                 law="bernoulli"):
        self.dims, self.B, self.L = list(dims), B, len(dims) - 1
        self._dims = (C.c_int64 * len(dims))(*dims)
        self.desc = rad_mlp_desc(self.L, ACTS[act], DTYPES[dtype], VARIANTS[variant], self._dims, B, p, 0, 0,
                                 LAWS[law])
        nbytes = C.c_int64(0)
        self.stats = rad_step_stats()
        _check(lib().rad_mlp_workspace(C.byref(self.desc), C.byref(nbytes), C.byref(self.stats)),
               "rad_mlp_workspace")
        self.workspace = torch.empty(nbytes.value, dtype=torch.uint8, device=device)
        self.dW = [torch.empty(dims[l], dims[l + 1], dtype=torch.float32, device=device) for l in range(self.L)]
        self.db = [torch.empty(dims[l + 1], dtype=torch.float32, device=device) for l in range(self.L)]
        self.loss = torch.zeros(1, dtype=torch.float32, device=device)
        self.nnz = torch.zeros(2 * self.L, dtype=torch.int64, device=device)
        self.dev_status = torch.zeros(1, dtype=torch.int32, device=device)
        arr = C.c_void_p * self.L
        self._dW = arr(*[t.data_ptr() for t in self.dW])
        self._db = arr(*[t.data_ptr() for t in self.db])

    def __call__(self, X, labels, Ws, bs, seed=0, step=0):
        return rad_mlp_step(self, X, labels, Ws, bs, seed, step)


def rad_mlp_step(ctx, X, labels, Ws, bs, seed=0, step=0):
    ctx.desc.seed, ctx.desc.step = seed, step
    arr = C.c_void_p * ctx.L
    W = arr(*[w.data_ptr() for w in Ws])
    b = arr(*[(None if t is None else t.data_ptr()) for t in bs])
    _check(lib().rad_mlp_step(C.byref(ctx.desc), _ptr(X), _ptr(labels), W, b, ctx._dW, ctx._db,
                              _ptr(ctx.loss), _ptr(ctx.nnz), _ptr(ctx.workspace), ctx.workspace.numel(),
                              _ptr(ctx.dev_status), _stream()), "rad_mlp_step")
    return ctx


class IRNNStep:
    """Owns the workspace and gradient buffers of rad_irnn_step for one shape."""

    def __init__(self, B, T, hidden, classes, variant="different", p=0.1, device="cuda"):
        self.desc = rad_irnn_desc(B, T, hidden, classes, VARIANTS[variant], p, 0, 0)
        nbytes = C.c_int64(0)
        self.stats = rad_step_stats()
        _check(lib().rad_irnn_workspace(C.byref(self.desc), C.byref(nbytes), C.byref(self.stats)), "rad_irnn_workspace")
        f32 = dict(dtype=torch.float32, device=device)
        self.workspace = torch.empty(nbytes.value, dtype=torch.uint8, device=device)
        self.dW_ih, self.db = torch.empty(hidden, **f32), torch.empty(hidden, **f32)
        self.dW_hh, self.dW_out = torch.empty(hidden, hidden, **f32), torch.empty(hidden, classes, **f32)
        self.db_out, self.loss = torch.empty(classes, **f32), torch.zeros(1, **f32)
        self.nnz = torch.zeros(2, dtype=torch.int64, device=device)
        self.dev_status = torch.zeros(1, dtype=torch.int32, device=device)

    def __call__(self, x, labels, W_ih, b_ih, W_hh, b_hh, W_out, b_out, seed=0, step0=0):
        return rad_irnn_step(self, x, labels, W_ih, b_ih, W_hh, b_hh, W_out, b_out, seed, step0)


def rad_irnn_step(ctx, x, labels, W_ih, b_ih, W_hh, b_hh, W_out, b_out, seed=0, step0=0):
    ctx.desc.seed, ctx.desc.step0 = seed, step0
    _check(lib().rad_irnn_step(C.byref(ctx.desc), _ptr(x), _ptr(labels), _ptr(W_ih), _ptr(b_ih), _ptr(W_hh),
                               _ptr(b_hh), _ptr(W_out), _ptr(b_out), _ptr(ctx.dW_ih), _ptr(ctx.db), _ptr(ctx.dW_hh),
                               _ptr(ctx.dW_out), _ptr(ctx.db_out), _ptr(ctx.loss), _ptr(ctx.nnz), _ptr(ctx.workspace),
                               ctx.workspace.numel(), _ptr(ctx.dev_status), _stream()), "rad_irnn_step")
    return ctx


class CNNStep:
    """Owns the workspace, gradient buffers and pointer tables of rad_cnn_step for one net shape."""

    def __init__(self, B, hw, cin, channels, fc, dtype="bf16", variant="different", p=0.1, device="cuda"):
        self.channels, self.fc = list(channels), list(fc)
        self._ch = (C.c_int64 * len(channels))(*channels)
        self._fc = (C.c_int64 * len(fc))(*fc)
        self.desc = rad_cnn_desc(B, hw, hw, cin, len(channels), len(fc), self._ch, self._fc, DTYPES[dtype],
                                 VARIANTS[variant], p, 0, 0)
        nbytes = C.c_int64(0)
        self.stats = rad_step_stats()
        _check(lib().rad_cnn_workspace(C.byref(self.desc), C.byref(nbytes), C.byref(self.stats)), "rad_cnn_workspace")
        f32 = dict(dtype=torch.float32, device=device)
        self.workspace = torch.empty(nbytes.value, dtype=torch.uint8, device=device)
        cs = [cin] + self.channels
        self.dconv_W = [torch.empty(3, 3, cs[l], cs[l + 1], **f32) for l in range(len(channels))]
        self.dconv_b = [torch.empty(cs[l + 1], **f32) for l in range(len(channels))]
        fs = [(hw >> len(channels)) ** 2 * cs[-1]] + self.fc
        self.dfc_W = [torch.empty(fs[l], fs[l + 1], **f32) for l in range(len(fc))]
        self.dfc_b = [torch.empty(fs[l + 1], **f32) for l in range(len(fc))]
        self.loss = torch.zeros(1, **f32)
        self.nnz = torch.zeros(2 * (len(channels) + len(fc)), dtype=torch.int64, device=device)
        self.dev_status = torch.zeros(1, dtype=torch.int32, device=device)

    def __call__(self, X, labels, conv_W, conv_b, fc_W, fc_b, seed=0, step=0):
        return rad_cnn_step(self, X, labels, conv_W, conv_b, fc_W, fc_b, seed, step)


def _table(tensors):
    return (C.c_void_p * len(tensors))(*[(None if t is None else t.data_ptr()) for t in tensors])


def rad_cnn_step(ctx, X, labels, conv_W, conv_b, fc_W, fc_b, seed=0, step=0):
    ctx.desc.seed, ctx.desc.step = seed, step
    _check(lib().rad_cnn_step(C.byref(ctx.desc), _ptr(X), _ptr(labels), _table(conv_W), _table(conv_b), _table(fc_W),
                              _table(fc_b), _table(ctx.dconv_W), _table(ctx.dconv_b), _table(ctx.dfc_W),
                              _table(ctx.dfc_b), _ptr(ctx.loss), _ptr(ctx.nnz), _ptr(ctx.workspace),
                              ctx.workspace.numel(), _ptr(ctx.dev_status), _stream()), "rad_cnn_step")
    return ctx
