"""ctypes binding of liblq.so: the same entry points as include/lq.h, taking torch tensors.

Only argument marshalling happens here (pointers, sizes, strides, dtypes).  Every step of
the pass runs in the library's CUDA kernels; if the library cannot be loaded, or a call
fails, an exception is raised -- there is no fallback path."""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# LQ_LIBRARY_VARIANT=debug selects the build with address checks in the kernels (liblq_debug.so, see build.py)
_LIB_PATH = os.path.join(_HERE, "liblq_debug.so" if os.environ.get("LQ_LIBRARY_VARIANT") == "debug" else "liblq.so")
_lib = None

LQ_F32, LQ_BF16 = 0, 1
LQ_GRID_NONUNIFORM, LQ_GRID_AFFINE = 0, 1
STATUS_NAMES = {0: "LQ_OK", 1: "LQ_ERR_INVALID_ARG", 2: "LQ_ERR_UNSUPPORTED", 3: "LQ_ERR_WORKSPACE_TOO_SMALL",
                4: "LQ_ERR_NOT_POSITIVE_DEFINITE", 5: "LQ_ERR_NONFINITE", 6: "LQ_ERR_CUDA", 7: "LQ_ERR_TIMEOUT",
                8: "LQ_ERR_STATIC_SCRATCH_TOO_SMALL"}


class LQError(RuntimeError):
    def __init__(self, code, where, info=None):
        self.code, self.info = code, info
        extra = f" (info={info})" if info is not None else ""
        super().__init__(f"{where}: {STATUS_NAMES.get(code, code)}{extra}")


class Config(C.Structure):
    """Mirror of lq_config."""
    _fields_ = [("bits", C.c_int32), ("grid_type", C.c_int32), ("p", C.c_float), ("n_iter", C.c_int32),
                ("init", C.c_int32), ("group_size", C.c_int32), ("T", C.c_int32), ("t_count", C.c_int32),
                ("block", C.c_int32), ("reserved", C.c_int32)]

    @classmethod
    def make(cls, grid="nonuniform", bits=4, p=4.0, n_iter=20, group=0, T=2048, t=None, block=128, init="uniform", **_):
        if t is None:
            t = int({4: 0.2, 3: 0.3, 2: 0.4}.get(bits, 0.2) * T)
        gt = LQ_GRID_NONUNIFORM if grid == "nonuniform" else LQ_GRID_AFFINE
        return cls(bits, gt, float(p), n_iter, {"uniform": 0, "weighted_quantile": 1}[init], group or 0, T, t, block, 0)


def library_path() -> str:
    return _LIB_PATH


def LQ():
    """The loaded library (loads it on first use; raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise LQError(6, f"liblq.so not built at {_LIB_PATH} (run paper_2407_10032_b200/build.py)")
        lib = C.CDLL(_LIB_PATH)
        vp, i32, i64, f32, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t
        P = C.POINTER
        sig = {
            "lq_create": [P(vp), C.c_int],
            "lq_destroy": [vp],
            "lq_sync_status": [vp, vp, P(i32), P(i64)],
            "lq_hessian_workspace": [i32, i32, i64, i64, P(sz)],
            "lq_hessian_accumulate": [vp, vp, vp, i32, i32, i64, i64, i64, vp, i64, f32, vp, sz],
            "lq_hessian_finalize": [vp, vp, vp, i64, i64],
            "lq_prepare_hinv_workspace": [i64, P(sz)],
            "lq_prepare_hinv": [vp, vp, vp, i64, i64, f32, vp, i64, vp, vp, i32, i64, i64, vp, sz],
            "lq_chol_diag": [vp, vp, vp, i64, i64, vp],
            "lq_fit_grid_workspace": [P(Config), i64, i64, P(sz)],
            "lq_fit_grid": [vp, vp, P(Config), vp, i32, i64, i64, i64, vp, vp, vp, vp, vp, sz],
            "lq_fit_grid_noalloc": [vp, vp, P(Config), vp, i32, i64, i64, i64, vp, vp, vp, vp],
            "lq_pack_codes": [vp, vp, vp, i64, i64, i32, vp, i64],
            "lq_peak_probe": [vp, vp, i32, i64, P(C.c_double)],
            "lq_pack_layer_bytes": [P(Config), i64, i64, P(sz), P(C.c_double)],
            "lq_pack_layer": [vp, vp, P(Config), vp, i64, i64, vp, vp, vp, vp, sz],
            "lq_unpack_layer": [vp, vp, P(Config), vp, sz, i64, i64, vp, i32, i64],
            "lq_zero_dead_columns": [vp, vp, vp, i64, i64, vp, i32, i64, i64],
            "lq_act_order": [vp, vp, vp, i64, i64, vp],
            "lq_permute_hessian": [vp, vp, vp, i64, i64, vp, vp, i64],
            "lq_gather_columns": [vp, vp, vp, i32, i64, i64, i64, vp, vp, i64],
            "lq_scatter_columns": [vp, vp, vp, i32, i64, i64, i64, vp, vp, i64],
            "lq_testing_set_wait_limit_ns": [vp, C.c_uint64],
            "lq_testing_inject_stall": [vp, i32],
            "lq_testing_set_prepare_defer_min_blocks": [vp, i32],
            "lq_testing_set_prepare_slices_int8": [vp, i32],
            "lq_quantize_layer_lazy_workspace": [P(Config), i64, i64, P(sz)],
            "lq_quantize_layer_lazy": [vp, vp, P(Config), vp, i32, i64, i64, i64, vp, i64, vp, vp, vp, vp, vp, i32, i64,
                                       vp, vp, sz],
            "lq_quantize_exact_workspace": [P(Config), i64, i64, P(sz)],
            "lq_quantize_exact": [vp, vp, P(Config), vp, i32, i64, i64, i64, vp, i64, vp, vp, vp, vp, vp, i32, i64,
                                  vp, vp, sz],
            "lq_quantize_layer_workspace": [P(Config), i64, i64, P(sz)],
            "lq_quantize_layer": [vp, vp, P(Config), vp, i32, i64, i64, i64, vp, i64, vp, vp, vp, vp, vp, i32, i64,
                                  vp, vp, sz],
        }
        for name, args in sig.items():
            fn = getattr(lib, name)
            fn.argtypes = args
            fn.restype = C.c_int
        lib.lq_launch_count.restype = C.c_uint64
        lib.lq_launch_count.argtypes = []
        lib.lq_version.restype = C.c_char_p
        lib.lq_version.argtypes = []
        _lib = lib
    return _lib


def _check(code, where):
    if code != 0:
        raise LQError(code, where)


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return LQ_F32
    if t.dtype == torch.bfloat16:
        return LQ_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _rowmajor(t: torch.Tensor):
    assert t.dim() == 2 and t.stride(1) == 1, "row-major 2-D tensor expected"
    return t.stride(0)


def lq_version() -> str:
    return LQ().lq_version().decode()


def lq_launch_count() -> int:
    return int(LQ().lq_launch_count())


def lq_create(device: int = 0):
    h = C.c_void_p()
    _check(LQ().lq_create(C.byref(h), device), "lq_create")
    return h


def lq_destroy(h):
    _check(LQ().lq_destroy(h), "lq_destroy")


def lq_sync_status(h, stream=None, raise_on_error=True):
    st, info = C.c_int32(0), C.c_int64(0)
    _check(LQ().lq_sync_status(h, _stream(stream), C.byref(st), C.byref(info)), "lq_sync_status")
    if st.value and raise_on_error:
        raise LQError(st.value, "device status", info.value)
    return st.value, info.value


def lq_hessian_workspace(x_dtype, c, n_chunk, token_major=False) -> int:
    b = C.c_size_t(0)
    dt = x_dtype if isinstance(x_dtype, int) else (LQ_F32 if x_dtype == torch.float32 else LQ_BF16)
    _check(LQ().lq_hessian_workspace(dt, 1 if token_major else 0, c, n_chunk, C.byref(b)), "lq_hessian_workspace")
    return b.value


def lq_hessian_accumulate(h, X, H, alpha=2.0, ws=None, stream=None, token_major=False):
    """X is c x n (feature-major) or, with token_major, n x c."""
    c, n = (X.shape[1], X.shape[0]) if token_major else X.shape
    _check(LQ().lq_hessian_accumulate(h, _stream(stream), _ptr(X), _dt(X), 1 if token_major else 0, c, n, _rowmajor(X), _ptr(H),
                                      _rowmajor(H), alpha, _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size()),
           "lq_hessian_accumulate")


def lq_hessian_finalize(h, H, stream=None):
    _check(LQ().lq_hessian_finalize(h, _stream(stream), _ptr(H), H.shape[0], _rowmajor(H)), "lq_hessian_finalize")


def lq_prepare_hinv_workspace(c) -> int:
    b = C.c_size_t(0)
    _check(LQ().lq_prepare_hinv_workspace(c, C.byref(b)), "lq_prepare_hinv_workspace")
    return b.value


def lq_prepare_hinv(h, H, U, dinv, ws, damp_frac=0.01, W=None, stream=None):
    c = H.shape[0]
    r, ldw, wdt = (0, 0, 0) if W is None else (W.shape[0], _rowmajor(W), _dt(W))
    _check(LQ().lq_prepare_hinv(h, _stream(stream), _ptr(H), c, _rowmajor(H), damp_frac, _ptr(U), _rowmajor(U),
                                _ptr(dinv), _ptr(W), wdt, r, ldw, _ptr(ws), ws.numel() * ws.element_size()),
           "lq_prepare_hinv")


def lq_chol_diag(h, U, d=None, stream=None):
    """Diagonal of the factor U, for the variant of the grid objective weighted by diag(U)^-p."""
    c = U.shape[0]
    if d is None:
        d = torch.empty((c,), dtype=torch.float32, device=U.device)
    _check(LQ().lq_chol_diag(h, _stream(stream), _ptr(U), c, _rowmajor(U), _ptr(d)), "lq_chol_diag")
    return d


def lq_fit_grid_workspace(cfg, r, c) -> int:
    b = C.c_size_t(0)
    _check(LQ().lq_fit_grid_workspace(C.byref(cfg), r, c, C.byref(b)), "lq_fit_grid_workspace")
    return b.value


def lq_fit_grid(h, cfg, W, dinv, ws, grid=None, scale=None, zero=None, stream=None):
    r, c = W.shape
    _check(LQ().lq_fit_grid(h, _stream(stream), C.byref(cfg), _ptr(W), _dt(W), r, c, _rowmajor(W), _ptr(dinv),
                            _ptr(grid), _ptr(scale), _ptr(zero), _ptr(ws), ws.numel() * ws.element_size()),
           "lq_fit_grid")


def lq_fit_grid_noalloc(h, cfg, W, dinv, grid=None, scale=None, zero=None, stream=None):
    """lq_fit_grid without a workspace: the scratch is an array built into the library, for callers
    that must not allocate device memory.  `h` may be None."""
    r, c = W.shape
    _check(LQ().lq_fit_grid_noalloc(h, _stream(stream), C.byref(cfg), _ptr(W), _dt(W), r, c, _rowmajor(W), _ptr(dinv),
                                    _ptr(grid), _ptr(scale), _ptr(zero)), "lq_fit_grid_noalloc")


def lq_quantize_layer_workspace(cfg, r, c) -> int:
    b = C.c_size_t(0)
    _check(LQ().lq_quantize_layer_workspace(C.byref(cfg), r, c, C.byref(b)), "lq_quantize_layer_workspace")
    return b.value


def lq_quantize_layer(h, cfg, W, U, codes, ws, grid=None, scale=None, zero=None, W_hat=None, loss_out=None, stream=None):
    r, c = W.shape
    whdt, ldwh = (0, 0) if W_hat is None else (_dt(W_hat), _rowmajor(W_hat))
    _check(LQ().lq_quantize_layer(h, _stream(stream), C.byref(cfg), _ptr(W), _dt(W), r, c, _rowmajor(W), _ptr(U),
                                  _rowmajor(U), _ptr(grid), _ptr(scale), _ptr(zero), _ptr(codes), _ptr(W_hat), whdt,
                                  ldwh, _ptr(loss_out), _ptr(ws), ws.numel() * ws.element_size()),
           "lq_quantize_layer")


def lq_quantize_layer_lazy_workspace(cfg, r, c) -> int:
    b = C.c_size_t(0)
    _check(LQ().lq_quantize_layer_lazy_workspace(C.byref(cfg), r, c, C.byref(b)), "lq_quantize_layer_lazy_workspace")
    return b.value


def lq_quantize_layer_lazy(h, cfg, W, U, dinv, scale, zero, codes, ws, W_hat=None, loss_out=None, stream=None):
    """lq_quantize_layer with each group's (S, Z) fitted when the column loop reaches the group (outputs scale, zero)."""
    r, c = W.shape
    whdt, ldwh = (0, 0) if W_hat is None else (_dt(W_hat), _rowmajor(W_hat))
    _check(LQ().lq_quantize_layer_lazy(h, _stream(stream), C.byref(cfg), _ptr(W), _dt(W), r, c, _rowmajor(W), _ptr(U),
                                       _rowmajor(U), _ptr(dinv), _ptr(scale), _ptr(zero), _ptr(codes), _ptr(W_hat), whdt,
                                       ldwh, _ptr(loss_out), _ptr(ws), ws.numel() * ws.element_size()),
           "lq_quantize_layer_lazy")


def lq_quantize_exact_workspace(cfg, r, c) -> int:
    b = C.c_size_t(0)
    _check(LQ().lq_quantize_exact_workspace(C.byref(cfg), r, c, C.byref(b)), "lq_quantize_exact_workspace")
    return b.value


def lq_quantize_exact(h, cfg, W, U, codes, ws, grid=None, scale=None, zero=None, W_hat=None, loss_out=None, stream=None):
    """Algorithm 2: greedy order and a full downdate of the inverse per row (small layers)."""
    r, c = W.shape
    whdt, ldwh = (0, 0) if W_hat is None else (_dt(W_hat), _rowmajor(W_hat))
    _check(LQ().lq_quantize_exact(h, _stream(stream), C.byref(cfg), _ptr(W), _dt(W), r, c, _rowmajor(W), _ptr(U),
                                  _rowmajor(U), _ptr(grid), _ptr(scale), _ptr(zero), _ptr(codes), _ptr(W_hat), whdt,
                                  ldwh, _ptr(loss_out), _ptr(ws), ws.numel() * ws.element_size()),
           "lq_quantize_exact")


def lq_peak_probe(h, kind, iters, stream=None) -> float:
    """Launches the dependent-free loop `kind` ("f32_fma", "f64_fma" or "f64_mma"); returns the operations it executes."""
    ops = C.c_double(0.0)
    k = {"f32_fma": 0, "f64_fma": 1, "f64_mma": 2}[kind]
    _check(LQ().lq_peak_probe(h, _stream(stream), k, iters, C.byref(ops)), "lq_peak_probe")
    return ops.value


def lq_testing_set_wait_limit_ns(h, ns):
    """Test hook (include/lq_testing.h): time limit of the bounded waits inside kernels; 0 restores the default."""
    _check(LQ().lq_testing_set_wait_limit_ns(h, ns), "lq_testing_set_wait_limit_ns")


def lq_testing_inject_stall(h, on):
    """Test hook (include/lq_testing.h): load barriers of the tensor-core contraction that never complete."""
    _check(LQ().lq_testing_inject_stall(h, 1 if on else 0), "lq_testing_inject_stall")


def lq_testing_set_prepare_defer_min_blocks(h, n_blocks):
    """Test hook (include/lq_testing.h): matrix size from which stage 2 defers far updates to the bf16 tensor cores."""
    _check(LQ().lq_testing_set_prepare_defer_min_blocks(h, n_blocks), "lq_testing_set_prepare_defer_min_blocks")


def lq_testing_set_prepare_slices_int8(h, on):
    """Test hook (include/lq_testing.h): digit slices of stage 2's deferred updates as 8-bit integers (default) or bf16."""
    _check(LQ().lq_testing_set_prepare_slices_int8(h, 1 if on else 0), "lq_testing_set_prepare_slices_int8")


def lq_pack_codes(h, codes, bits, packed=None, stream=None):
    """b-bit little-endian packing of the one-code-per-byte output; returns the packed tensor."""
    r, c = codes.shape
    nbytes = (c * bits + 7) // 8
    if packed is None:
        packed = torch.empty((r, nbytes), dtype=torch.uint8, device=codes.device)
    _check(LQ().lq_pack_codes(h, _stream(stream), _ptr(codes), r, c, bits, _ptr(packed), _rowmajor(packed)), "lq_pack_codes")
    return packed


def lq_pack_layer_bytes(cfg, r, c):
    """(bytes of a layer record, bits per weight of the format)."""
    b, bpw = C.c_size_t(0), C.c_double(0.0)
    _check(LQ().lq_pack_layer_bytes(C.byref(cfg), r, c, C.byref(b), C.byref(bpw)), "lq_pack_layer_bytes")
    return b.value, bpw.value


def lq_pack_layer(h, cfg, codes, grid=None, scale=None, zero=None, record=None, stream=None):
    """The layer as one record (packed codes + fp16 tables, or fp16 scales + int16 zero points); returns the record."""
    r, c = codes.shape
    nbytes, _ = lq_pack_layer_bytes(cfg, r, c)
    if record is None:
        record = torch.zeros((nbytes,), dtype=torch.uint8, device=codes.device)
    _check(LQ().lq_pack_layer(h, _stream(stream), C.byref(cfg), _ptr(codes), r, c, _ptr(grid), _ptr(scale), _ptr(zero),
                              _ptr(record), record.numel()), "lq_pack_layer")
    return record


def lq_unpack_layer(h, cfg, record, r, c, W_hat=None, dtype=torch.float32, stream=None):
    """The weights a record stands for."""
    if W_hat is None:
        W_hat = torch.empty((r, c), dtype=dtype, device=record.device)
    _check(LQ().lq_unpack_layer(h, _stream(stream), C.byref(cfg), _ptr(record), record.numel(), r, c, _ptr(W_hat), _dt(W_hat),
                                _rowmajor(W_hat)), "lq_unpack_layer")
    return W_hat


def lq_zero_dead_columns(h, H, W, stream=None):
    """Zeroes the columns of W whose input channel never fired (H_ii = 0): for layers that share a Hessian."""
    r, c = W.shape
    _check(LQ().lq_zero_dead_columns(h, _stream(stream), _ptr(H), c, _rowmajor(H), _ptr(W), _dt(W), r, _rowmajor(W)),
           "lq_zero_dead_columns")


def lq_act_order(h, H, perm=None, stream=None):
    """perm[k] = the column taken k-th when columns go in the order of decreasing diag(H)."""
    c = H.shape[0]
    if perm is None:
        perm = torch.empty((c,), dtype=torch.int32, device=H.device)
    _check(LQ().lq_act_order(h, _stream(stream), _ptr(H), c, _rowmajor(H), _ptr(perm)), "lq_act_order")
    return perm


def lq_permute_hessian(h, H, perm, Hp, stream=None):
    c = H.shape[0]
    _check(LQ().lq_permute_hessian(h, _stream(stream), _ptr(H), c, _rowmajor(H), _ptr(perm), _ptr(Hp), _rowmajor(Hp)),
           "lq_permute_hessian")


def lq_gather_columns(h, src, perm, dst, stream=None):
    r, c = src.shape
    _check(LQ().lq_gather_columns(h, _stream(stream), _ptr(src), src.element_size(), r, c, _rowmajor(src), _ptr(perm), _ptr(dst),
                                  _rowmajor(dst)), "lq_gather_columns")


def lq_scatter_columns(h, src, perm, dst, stream=None):
    r, c = src.shape
    _check(LQ().lq_scatter_columns(h, _stream(stream), _ptr(src), src.element_size(), r, c, _rowmajor(src), _ptr(perm), _ptr(dst),
                                   _rowmajor(dst)), "lq_scatter_columns")


class StackPass:
    """A stack of layers quantised in order, the way a model-level driver walks a decoder block: layers that read the
    same activations form a group and share stages 1-2 (one Hessian, one factor); every layer then gets its own grid,
    its column loop and its packed record.  Only buffers and the order of the library calls live here.

    groups: list of (c, [r, ...]) -- input width of the group and the output widths of its layers."""

    def __init__(self, handle, groups, cfg: Config, w_dtype=torch.bfloat16, x_dtype=torch.bfloat16, n_chunk=0,
                 device="cuda", want_w_hat=False, want_records=True):
        self.h, self.cfg, self.groups, self.want_records = handle, cfg, groups, want_records
        self.passes = []
        for c, rs in groups:
            ps = []
            for r in rs:                          # one Hessian, one factor and one inverse diagonal per group
                ps.append(LayerPass(handle, r, c, cfg, w_dtype=w_dtype, x_dtype=x_dtype, n_chunk=n_chunk, device=device,
                                    want_w_hat=want_w_hat, share=ps[0] if ps else None))
            self.passes.append(ps)
        self.records = [[None] * len(rs) for _, rs in groups]

    def run(self, inputs, weights, damp_frac=0.01, alpha=2.0, n_chunk=0, on_layer=None):
        """inputs[g]: the group's activations X (c x n); weights[g][l]: that layer's W (r x c, dead columns are zeroed
        in place).  `on_layer(g, l)` is called after each layer's work has been enqueued (a benchmark records an event)."""
        for g, (X, Ws, ps) in enumerate(zip(inputs, weights, self.passes)):
            P0 = ps[0]
            n = X.shape[1]
            step = n if n_chunk <= 0 else n_chunk
            P0.H.zero_()
            for j in range(0, n, step):
                lq_hessian_accumulate(self.h, X[:, j:j + step], P0.H, alpha, P0.ws)
            lq_hessian_finalize(self.h, P0.H)
            lq_prepare_hinv(self.h, P0.H, P0.U, P0.dinv, P0.ws, damp_frac, Ws[0])
            for W in Ws[1:]:
                lq_zero_dead_columns(self.h, P0.H, W)
            if on_layer:
                on_layer(g, -1)
            for l, (W, P) in enumerate(zip(Ws, ps)):
                lq_fit_grid(self.h, self.cfg, W, P0.dinv, P.ws, P.grid, P.scale, P.zero)
                lq_quantize_layer(self.h, self.cfg, W, P0.U, P.codes, P.ws, P.grid, P.scale, P.zero, P.W_hat, P.loss)
                if self.want_records:
                    self.records[g][l] = lq_pack_layer(self.h, self.cfg, P.codes, P.grid, P.scale, P.zero, self.records[g][l])
                if on_layer:
                    on_layer(g, l)


class LayerPass:
    """Buffers for one layer shape plus the four calls in Algorithm 1's order.

    Allocation only (through torch's allocator); all arithmetic is in liblq."""

    def __init__(self, handle, r, c, cfg: Config, w_dtype=torch.bfloat16, x_dtype=torch.bfloat16, n_chunk=0,
                 device="cuda", want_w_hat=True, weight_src="inv_diag", share=None, act_order=False):
        if weight_src not in ("inv_diag", "chol_diag"):
            raise ValueError("weight_src: 'inv_diag' (Eq. 5 / Eq. 7) or 'chol_diag' (Algorithm 1 to the letter)")
        self.weight_src = weight_src
        self.h, self.r, self.c, self.cfg = handle, r, c, cfg
        dev = torch.device(device)
        self.act_order = act_order
        if act_order:                         # the pass runs on the permuted layer: its inputs and outputs in that order
            self.perm = torch.empty((c,), dtype=torch.int32, device=dev)
            self.Wp = torch.empty((r, c), dtype=w_dtype, device=dev)
            self.codes_p = torch.empty((r, c), device=dev, dtype=torch.uint8)
            self.W_hat_p = torch.empty((r, c), device=dev, dtype=w_dtype) if want_w_hat else None
        K = 1 << cfg.bits
        f32 = dict(device=dev, dtype=torch.float32)
        if share is not None:                 # a layer that reads the same activations: one Hessian, factor and diagonal
            self.H, self.U, self.dinv = share.H, share.U, share.dinv
        else:
            self.H = torch.zeros((c, c), **f32)
            self.U = torch.empty((c, c), **f32)
            self.dinv = torch.empty((c,), **f32)
        self.affine = cfg.grid_type == LQ_GRID_AFFINE
        ng = 1 if cfg.group_size == 0 else c // cfg.group_size
        self.grid = None if self.affine else torch.empty((r, K), **f32)
        self.scale = torch.empty((r, ng), **f32) if self.affine else None
        self.zero = torch.empty((r, ng), device=dev, dtype=torch.int32) if self.affine else None
        self.codes = torch.empty((r, c), device=dev, dtype=torch.uint8)
        self.W_hat = torch.empty((r, c), device=dev, dtype=w_dtype) if want_w_hat else None
        self.loss = torch.zeros((1,), device=dev, dtype=torch.float64)
        nbytes = max(lq_hessian_workspace(x_dtype, c, n_chunk), lq_prepare_hinv_workspace(c),
                     lq_fit_grid_workspace(cfg, r, c), lq_quantize_layer_workspace(cfg, r, c), 256)
        self.ws = torch.empty((nbytes,), device=dev, dtype=torch.uint8)

    def accumulate(self, X, alpha=2.0):
        lq_hessian_accumulate(self.h, X, self.H, alpha, self.ws)

    def finish(self, W, damp_frac=0.01):
        """Stages 2-4 after all chunks were accumulated."""
        lq_hessian_finalize(self.h, self.H)
        if self.act_order:
            # columns in the order of decreasing diag(H): H permuted into U's buffer (stage 2 may run in place there),
            # W gathered, the pass as usual, codes and W_hat scattered back
            lq_act_order(self.h, self.H, self.perm)
            lq_permute_hessian(self.h, self.H, self.perm, self.U)
            lq_gather_columns(self.h, W, self.perm, self.Wp)
            lq_prepare_hinv(self.h, self.U, self.U, self.dinv, self.ws, damp_frac, self.Wp)
            if self.weight_src == "chol_diag":
                lq_chol_diag(self.h, self.U, self.dinv)
            lq_fit_grid(self.h, self.cfg, self.Wp, self.dinv, self.ws, self.grid, self.scale, self.zero)
            lq_quantize_layer(self.h, self.cfg, self.Wp, self.U, self.codes_p, self.ws, self.grid, self.scale, self.zero,
                              self.W_hat_p, self.loss)
            lq_scatter_columns(self.h, self.codes_p, self.perm, self.codes)
            if self.W_hat is not None:
                lq_scatter_columns(self.h, self.W_hat_p, self.perm, self.W_hat)
            return
        lq_prepare_hinv(self.h, self.H, self.U, self.dinv, self.ws, damp_frac, W)
        if self.weight_src == "chol_diag":
            lq_chol_diag(self.h, self.U, self.dinv)
        lq_fit_grid(self.h, self.cfg, W, self.dinv, self.ws, self.grid, self.scale, self.zero)
        lq_quantize_layer(self.h, self.cfg, W, self.U, self.codes, self.ws, self.grid, self.scale, self.zero,
                          self.W_hat, self.loss)

    def run(self, W, X, damp_frac=0.01, alpha=2.0):
        self.H.zero_()
        self.accumulate(X, alpha)
        self.finish(W, damp_frac)

    def accumulate_from_host(self, chunks, alpha=2.0):
        """Stage 1 for calibration activations that live in pinned host memory as a sequence of contiguous
        chunks (each c x m_i, tokens contiguous): every chunk is copied to one of two device staging buffers
        on a side stream while the previous chunk is being accumulated, so the copy and the contraction
        overlap.  Plumbing only (copies, streams, events); the arithmetic is lq_hessian_accumulate's."""
        chunks = list(chunks)
        if not chunks:
            return
        c = chunks[0].shape[0]
        widest = max(t.shape[1] for t in chunks)
        dev = self.H.device
        main = torch.cuda.current_stream(dev)
        if getattr(self, "_stage", None) is None or self._stage[0].shape[1] < widest or self._stage[0].dtype != chunks[0].dtype:
            self._stage = [torch.empty((c, widest), dtype=chunks[0].dtype, device=dev) for _ in range(2)]
            self._copy_stream = torch.cuda.Stream(dev)
            self._filled = [torch.cuda.Event() for _ in range(2)]
            self._drained = [torch.cuda.Event() for _ in range(2)]
        self._copy_stream.wait_stream(main)            # earlier work on the staging buffers has finished
        for k, Xc in enumerate(chunks):
            b = k & 1
            m = Xc.shape[1]
            dst = self._stage[b].view(-1)[:c * m].view(c, m)       # contiguous c x m inside the staging buffer
            with torch.cuda.stream(self._copy_stream):
                if k >= 2:
                    self._copy_stream.wait_event(self._drained[b])
                dst.copy_(Xc, non_blocking=True)
                self._filled[b].record(self._copy_stream)
            main.wait_event(self._filled[b])
            lq_hessian_accumulate(self.h, dst, self.H, alpha, self.ws)
            self._drained[b].record(main)
