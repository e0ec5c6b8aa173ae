"""ctypes binding over libmoonwalk.so: argument marshalling only.

Every step of the Moonwalk path runs inside the CUDA library; this module converts Python
objects (torch tensors used purely as device buffers) into the pointers and sizes of the C ABI
declared in include/moonwalk.h.  There is no CPU fallback: if the library is missing or a CUDA
device is absent, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmoonwalk.so")

MW_OK = 0
STATUS_NAMES = ["MW_OK", "MW_ERR_INVALID_ARG", "MW_ERR_UNSUPPORTED", "MW_ERR_WORKSPACE",
                "MW_ERR_STATE", "MW_ERR_NOT_SUBMERSIVE", "MW_ERR_TIMEOUT", "MW_ERR_CUDA"]
KIND = {"dense": 0, "conv2d": 1, "head": 2, "conv1d": 3}
ACT = {"none": 0, "leaky_relu": 1, "relu": 2}
PREC = {"f64": 0, "f32": 1, "bf16_f32acc": 2}
LOSS = {"half_sse": 0, "mse_mean": 1, "xent_mean": 2}
BACKEND = {"auto": 0, "simt": 1, "tensor": 2}


class MwError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        name = STATUS_NAMES[code] if 0 <= code < len(STATUS_NAMES) else str(code)
        super().__init__(f"{where}: {name}")


class LayerDesc(C.Structure):
    _fields_ = [("kind", C.c_int32), ("act", C.c_int32), ("slope", C.c_double),
                ("n_in", C.c_int32), ("n_out", C.c_int32), ("H", C.c_int32), ("W", C.c_int32),
                ("C_in", C.c_int32), ("C_out", C.c_int32), ("k", C.c_int32),
                ("stride", C.c_int32), ("pad", C.c_int32)]


class NetOpts(C.Structure):
    _fields_ = [("prec", C.c_int32), ("loss", C.c_int32), ("reseed_every", C.c_int32),
                ("conv_vijp_iters", C.c_int32), ("backend", C.c_int32),
                ("inverse_iters", C.c_int32), ("resident_inverse", C.c_int32),
                ("warm_inverse", C.c_int32), ("frag_block", C.c_int32), ("lu_param", C.c_int32)]


_lib = None


def lib() -> C.CDLL:
    """Load the CUDA library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_2402_14212_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
        L.mw_net_create.argtypes = [C.POINTER(LayerDesc), i32, i32, C.POINTER(NetOpts), C.POINTER(vp)]
        L.mw_net_destroy.argtypes = [vp]
        L.mw_net_destroy.restype = None
        L.mw_workspace_bytes.argtypes = [vp, C.POINTER(sz), C.POINTER(sz), C.POINTER(sz)]
        L.mw_input_cotangent.argtypes = [vp, C.POINTER(vp), vp, vp, vp, vp, vp, sz, vp]
        L.mw_forward_sweep.argtypes = [vp, C.POINTER(vp), vp, vp, C.POINTER(vp), vp, sz, vp]
        L.mw_forward_sweep_apply.argtypes = [vp, C.POINTER(vp), vp, vp, C.c_double, C.POINTER(vp), vp, sz, vp]
        L.mw_sweep_bucket_events.argtypes = [vp, i32, C.POINTER(vp), i32]
        L.mw_backprop_reference.argtypes = [vp, C.POINTER(vp), vp, vp, C.POINTER(vp), vp, vp, sz, vp]
        L.mw_export_masks.argtypes = [vp, vp, i32, vp, sz, C.POINTER(i32), C.POINTER(i32), vp]
        L.mw_last_device_status.argtypes = [vp, vp, vp, C.POINTER(C.c_uint32)]
        L.mw_status_string.argtypes = [i32]
        L.mw_status_string.restype = C.c_char_p
        L.mw_pack_sign_bits.argtypes = [vp, i32, i64, i32, vp, vp]
        L.mw_relu_fragment_compact.argtypes = [vp, vp, i64, i32, vp, vp, vp, vp, vp, sz, vp]
        L.mw_activation_vijp.argtypes = [vp, vp, i64, i32, i32, C.c_float, vp, vp, vp, vp, vp]
        L.mw_gemm_split_bf16.argtypes = [vp, i32, vp, i32, vp, i32, i32, i32, i32, vp, sz, vp]
        L.mw_conv2d_split_bf16.argtypes = [i32, vp, vp, vp, i32, i32, i32, i32, i32, vp, sz, vp]
        L.mw_conv2d_strided_split_bf16.argtypes = [i32, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32,
                                                   i32, vp, sz, vp]
        L.mw_gemm_split_bf16_static.argtypes = [vp, i32, vp, i32, vp, i32, i32, i32, i32, vp]
        L.mw_gradient_step_host.argtypes = [vp, C.POINTER(vp), vp, sz, vp, sz, vp, vp, vp,
                                            C.POINTER(vp), vp, vp, vp, sz, vp]
        L.mw_launch_count.argtypes = []
        L.mw_launch_count.restype = C.c_int64
        L.mw_set_pair_mode.argtypes = [i32]
        L.mw_set_pair_mode.restype = i32
        L.mw_selftest_bounded_wait.argtypes = [vp, sz, C.c_uint32, C.POINTER(i32), vp]
        L.mw_set_sweep_chains.argtypes = [i32]
        L.mw_set_sweep_chains.restype = i32
        L.mw_set_bulk_epilogue.argtypes = [i32]
        L.mw_set_bulk_epilogue.restype = i32
        L.mw_set_cooperative_launch.argtypes = [i32]
        L.mw_set_cooperative_launch.restype = i32
        L.mw_set_merge_orders.argtypes = [i32]
        L.mw_set_merge_orders.restype = i32
        L.mw_profile_begin.argtypes = []
        L.mw_profile_begin.restype = None
        L.mw_profile_end.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_int64),
                                     C.POINTER(C.c_double), C.POINTER(C.c_double)]
        _lib = L
    return _lib


def _check(code: int, where: str):
    if code != MW_OK:
        raise MwError(code, where)


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def _stream_handle(stream=None) -> int:
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _ptr_array(tensors: Sequence) -> "C.Array":
    arr = (C.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = _ptr(t)
    return arr


def make_layer_descs(layers) -> "C.Array":
    arr = (LayerDesc * len(layers))()
    for i, l in enumerate(layers):
        arr[i] = LayerDesc(KIND[l.kind], ACT[l.act], float(l.slope), int(l.n_in), int(l.n_out),
                           int(l.H), int(l.W), int(l.C_in), int(l.C_out), int(l.k),
                           int(l.stride), int(l.pad))
    return arr


class Net:
    """Host-side handle of one network (mw_net).  Owns no device memory."""

    def __init__(self, layers, batch: int, prec: str, loss: str, reseed_every: int = 4,
                 conv_vijp_iters: int = 10, backend: str = "auto", inverse_iters: int = 0,
                 resident_inverse: bool = True, frag_block: int = 0, warm_inverse: bool = False):
        self.layers = list(layers)
        # LU-parameterised dense layers (Layer.lu): all layers of a net or none
        lu = [bool(getattr(l, "lu", False)) for l in self.layers]
        if any(lu) and not all(lu):
            raise ValueError("a net is LU-parameterised in every layer or in none")
        self.batch = int(batch)
        self.prec, self.loss = prec, loss
        self._h = C.c_void_p()
        opts = NetOpts(PREC[prec], LOSS[loss], int(reseed_every), int(conv_vijp_iters),
                       BACKEND[backend], int(inverse_iters), int(bool(resident_inverse)),
                       int(bool(warm_inverse)), int(frag_block), int(any(lu)))
        descs = make_layer_descs(self.layers)
        _check(lib().mw_net_create(descs, len(self.layers), self.batch, C.byref(opts),
                                   C.byref(self._h)), "mw_net_create")

    def close(self):
        if self._h:
            lib().mw_net_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- sizes -------------------------------------------------------------------------
    def workspace_bytes(self):
        a, b = C.c_size_t(), C.c_size_t()
        res = (C.c_size_t * 2)()
        _check(lib().mw_workspace_bytes(self._h, C.byref(a), C.byref(b), res), "mw_workspace_bytes")
        return int(a.value), int(b.value), (int(res[0]), int(res[1]))

    def grad_dtype(self):
        import torch
        return torch.float64 if self.prec == "f64" else torch.float32

    def storage_dtype(self):
        import torch
        return {"f64": torch.float64, "f32": torch.float32, "bf16_f32acc": torch.bfloat16}[self.prec]

    def alloc_workspace(self, which: str = "moonwalk", device="cuda"):
        import torch
        a, b, _ = self.workspace_bytes()
        n = a if which == "moonwalk" else (b if which == "backprop" else max(a, b))
        return torch.empty(n + 256, dtype=torch.uint8, device=device)

    @staticmethod
    def _ws(workspace):
        p = int(workspace.data_ptr())
        ap = (p + 255) // 256 * 256
        return ap, workspace.numel() - (ap - p)

    # ---- the three calls ------------------------------------------------------------------
    def input_cotangent(self, params, x, target, workspace, g0_out=None, loss_out=None, stream=None,
                        keep_seed=False):
        """keep_seed (nets of strided submersive convolutions only): g0 is not returned; the part
        of it that the sweep reads stays in the workspace (call forward_sweep with g0 = None)."""
        import torch
        if g0_out is None and not keep_seed:
            g0_out = torch.empty(x.shape, dtype=self.grad_dtype(), device=x.device)
        wp, wb = self._ws(workspace)
        _check(lib().mw_input_cotangent(self._h, _ptr_array(params), _ptr(x), _ptr(target),
                                        _ptr(g0_out), _ptr(loss_out), wp, wb,
                                        _stream_handle(stream)), "mw_input_cotangent")
        return g0_out

    def forward_sweep(self, params, x, g0, workspace, dW_out=None, stream=None):
        import torch
        if dW_out is None:
            dW_out = [torch.empty(p.shape, dtype=self.grad_dtype(), device=p.device) for p in params]
        wp, wb = self._ws(workspace)
        _check(lib().mw_forward_sweep(self._h, _ptr_array(params), _ptr(x), _ptr(g0),
                                      _ptr_array(dW_out), wp, wb, _stream_handle(stream)),
               "mw_forward_sweep")
        return dW_out

    def forward_sweep_apply(self, params, x, g0, lr: float, workspace, params_out=None, stream=None):
        """theta_l <- theta_l - lr * g_l inside the sweep; in place unless `params_out` is given."""
        if params_out is None:
            params_out = params
        wp, wb = self._ws(workspace)
        _check(lib().mw_forward_sweep_apply(self._h, _ptr_array(params), _ptr(x), _ptr(g0), float(lr),
                                            _ptr_array(params_out), wp, wb, _stream_handle(stream)),
               "mw_forward_sweep_apply")
        return params_out

    def set_bucket_events(self, layers_per_bucket: int, events=None):
        """events: torch.cuda.Event objects (already recorded once, so that their handles exist), one
        per bucket of `layers_per_bucket` layers; the forward sweep records them as the buckets'
        gradients are enqueued.  layers_per_bucket = 0 turns the feature off."""
        events = list(events or [])
        arr = (C.c_void_p * max(1, len(events)))()
        for i, e in enumerate(events):
            arr[i] = int(e.cuda_event)
        _check(lib().mw_sweep_bucket_events(self._h, int(layers_per_bucket), arr, len(events)),
               "mw_sweep_bucket_events")
        self._bucket_events = events          # keep them alive

    def backprop_reference(self, params, x, target, workspace, dW_out=None, loss_out=None,
                           stream=None):
        import torch
        if dW_out is None:
            dW_out = [torch.empty(p.shape, dtype=self.grad_dtype(), device=p.device) for p in params]
        wp, wb = self._ws(workspace)
        _check(lib().mw_backprop_reference(self._h, _ptr_array(params), _ptr(x), _ptr(target),
                                           _ptr_array(dW_out), _ptr(loss_out), wp, wb,
                                           _stream_handle(stream)), "mw_backprop_reference")
        return dW_out

    def gradient_step_host(self, params, x_host, target_host, x_dev, target_dev, g0_dev, dW_out,
                           loss_dev, loss_host, workspace, stream=None):
        """Whole step with the per-step inputs in (pinned) host memory; returns after the loss
        has landed in `loss_host`."""
        wp, wb = self._ws(workspace)
        _check(lib().mw_gradient_step_host(
            self._h, _ptr_array(params), _ptr(x_host), x_host.numel() * x_host.element_size(),
            _ptr(target_host), target_host.numel() * target_host.element_size(), _ptr(x_dev),
            _ptr(target_dev), _ptr(g0_dev), _ptr_array(dW_out), _ptr(loss_dev), _ptr(loss_host),
            wp, wb, _stream_handle(stream)), "mw_gradient_step_host")

    def export_masks(self, workspace, layer: int, stream=None) -> np.ndarray:
        l = self.layers[layer]
        if l.kind in ("conv2d", "conv1d"):
            ho, wo = l.out_hw()
            rows, cols = self.batch * ho * wo, l.C_out
        else:
            rows, cols = self.batch, l.n_out
        wpr = (cols + 31) // 32
        out = np.zeros((rows, wpr), dtype=np.uint32)
        wp, _ = self._ws(workspace)
        r, w = C.c_int32(), C.c_int32()
        _check(lib().mw_export_masks(self._h, wp, layer, out.ctypes.data, out.size, C.byref(r),
                                     C.byref(w), _stream_handle(stream)), "mw_export_masks")
        assert (r.value, w.value) == (rows, wpr)
        return out

    def last_device_status(self, workspace, stream=None):
        wp, _ = self._ws(workspace)
        detail = (C.c_uint32 * 4)()
        code = lib().mw_last_device_status(self._h, wp, _stream_handle(stream), detail)
        return code, list(detail)


def launch_count() -> int:
    return int(lib().mw_launch_count())


def set_pair_mode(enable: bool) -> bool:
    """Turn the CTA-pair form of the product kernel on or off; returns the previous setting."""
    return bool(lib().mw_set_pair_mode(int(bool(enable))))


def selftest_bounded_wait(limit_ms: int = 5, stream=None) -> int:
    """Run the library's self-test of its bounded device-side waits; returns the status that the
    deliberately unsatisfiable launch recorded (MW_ERR_TIMEOUT = 6 when the path works)."""
    import torch
    scratch = torch.empty(512 * 1024, dtype=torch.uint8, device="cuda")
    p = (int(scratch.data_ptr()) + 255) // 256 * 256
    out = C.c_int32(-1)
    _check(lib().mw_selftest_bounded_wait(p, scratch.numel() - 256, int(limit_ms), C.byref(out),
                                          _stream_handle(stream)), "mw_selftest_bounded_wait")
    return int(out.value)


def set_sweep_chains(mode: int) -> int:
    """Forward sweep of dense nets as per-row-block chains in one launch (1: form chosen by tile
    count, 2: CTA pairs whenever possible) or as a launch per layer (0).  Returns the old mode."""
    return int(lib().mw_set_sweep_chains(int(mode)))


def set_bulk_epilogue(enable: bool) -> bool:
    """Epilogue outputs through the copy engine (True) or per-lane stores (False)."""
    return bool(lib().mw_set_bulk_epilogue(int(bool(enable))))


def set_cooperative_launch(enable: bool) -> bool:
    """Program launches with or without the cooperative-launch attribute (profiling aid)."""
    return bool(lib().mw_set_cooperative_launch(int(bool(enable))))


def set_merge_orders(enable: bool) -> bool:
    """Two-term products of the pair form: one accumulator block for all cross products (True) or
    one per order (False); returns the previous setting."""
    return bool(lib().mw_set_merge_orders(int(bool(enable))))


def profile_begin():
    lib().mw_profile_begin()


def profile_end():
    ms, n, fl, mfl = C.c_double(), C.c_int64(), C.c_double(), C.c_double()
    _check(lib().mw_profile_end(C.byref(ms), C.byref(n), C.byref(fl), C.byref(mfl)), "mw_profile_end")
    return dict(total_ms=ms.value, launches=int(n.value), flops=fl.value, mma_flops=mfl.value)


# ---- stand-alone kernels -----------------------------------------------------------------
def pack_sign_bits(z, words=None, stream=None):
    import torch
    dt = {torch.float64: 0, torch.float32: 1, torch.bfloat16: 2}[z.dtype]
    rows, cols = z.shape
    if words is None:
        words = torch.zeros((rows, (cols + 31) // 32), dtype=torch.int32, device=z.device)
    _check(lib().mw_pack_sign_bits(_ptr(z), dt, rows, cols, _ptr(words), _stream_handle(stream)),
           "mw_pack_sign_bits")
    return words


def relu_fragment_compact(h, words, stream=None):
    import torch
    rows, cols = h.shape
    dev = h.device
    cnt = torch.zeros(max(rows, 1), dtype=torch.int32, device=dev)
    off = torch.zeros(max(rows, 1), dtype=torch.int32, device=dev)
    vals = torch.zeros(max(rows * cols, 1), dtype=torch.float32, device=dev)
    total = torch.zeros(1, dtype=torch.int32, device=dev)
    scratch = torch.empty(4 * (rows + 1024), dtype=torch.uint8, device=dev)
    _check(lib().mw_relu_fragment_compact(_ptr(h), _ptr(words), rows, cols, _ptr(cnt), _ptr(off),
                                          _ptr(vals), _ptr(total), _ptr(scratch), scratch.numel(),
                                          _stream_handle(stream)), "mw_relu_fragment_compact")
    return cnt[:rows], off[:rows], vals, total


def activation_vijp(gz, words, act: str, slope: float = 0.0, off=None, vals=None, want_gz=False,
                    stream=None):
    import torch
    rows, cols = gz.shape
    h = torch.empty_like(gz)
    gzo = torch.empty_like(gz) if want_gz else None
    _check(lib().mw_activation_vijp(_ptr(gz), _ptr(words), rows, cols, ACT[act], float(slope),
                                    _ptr(off), _ptr(vals), _ptr(h), _ptr(gzo),
                                    _stream_handle(stream)), "mw_activation_vijp")
    return (h, gzo) if want_gz else h


def gemm_split_bf16(A, B, a_mn: bool, b_mn: bool, terms: int, stream=None):
    """D = op(A) op(B)^T-style product on the tensor cores (see moonwalk.h)."""
    import torch
    M = A.shape[1] if a_mn else A.shape[0]
    K = A.shape[0] if a_mn else A.shape[1]
    N = B.shape[1] if b_mn else B.shape[0]
    D = torch.empty((M, N), dtype=torch.float32, device=A.device)
    scratch = torch.empty(6 * (M * K + N * K) + 4096, dtype=torch.uint8, device=A.device)
    _check(lib().mw_gemm_split_bf16(_ptr(A), int(a_mn), _ptr(B), int(b_mn), _ptr(D), M, N, K,
                                    int(terms), _ptr(scratch), scratch.numel(),
                                    _stream_handle(stream)), "mw_gemm_split_bf16")
    return D


def conv2d_split_bf16(op: int, a, b, k: int, terms: int, stream=None):
    """op 0: conv(a = x, b = w); op 1: TransposeConv(a = h', b = w); op 2: weight vjp (a = x, b = g_z)."""
    import torch
    images, H, W, C = a.shape
    assert C == 64
    out = torch.empty((k, k, 64, 64) if op == 2 else (images, H, W, 64), dtype=torch.float32,
                      device=a.device)
    n = 1024 + 8 * terms * (a.numel() + b.numel()) + 256 * k * k * 16384 + 4096
    scratch = torch.empty(n, dtype=torch.uint8, device=a.device)
    _check(lib().mw_conv2d_split_bf16(op, _ptr(a), _ptr(b), _ptr(out), images, H, W, k, int(terms),
                                      _ptr(scratch), scratch.numel(), _stream_handle(stream)),
           "mw_conv2d_split_bf16")
    return out


def conv2d_strided_split_bf16(op: int, a, b, k: int, stride: int, pad: int, terms: int, in_hw=None,
                              stream=None):
    """op 0: conv(a = x, b = w); op 1: TransposeConv(a = h', b = w) back to the `in_hw` image;
    op 2: weight vjp (a = x, b = g_z).  Channel-last float tensors, C channels in and out."""
    import torch
    images, Ha, Wa, C = a.shape
    if op == 1:
        H, W = in_hw
    else:
        H, W = Ha, Wa
    Ho, Wo = (H + 2 * pad - k) // stride + 1, (W + 2 * pad - k) // stride + 1
    shape = {0: (images, Ho, Wo, C), 1: (images, H, W, C), 2: (k, k, C, C)}[op]
    out = torch.empty(shape, dtype=torch.float32, device=a.device)
    n = 1024 + 8 * terms * (a.numel() + b.numel()) + 1024 * k * k * C * C + 4096
    scratch = torch.empty(n, dtype=torch.uint8, device=a.device)
    _check(lib().mw_conv2d_strided_split_bf16(op, _ptr(a), _ptr(b), _ptr(out), images, H, W, C, k,
                                              stride, pad, int(terms), _ptr(scratch), scratch.numel(),
                                              _stream_handle(stream)),
           "mw_conv2d_strided_split_bf16")
    return out


GEMM_STATIC_SCRATCH_BYTES = 16 << 20


def gemm_split_bf16_static(A, B, a_mn: bool, b_mn: bool, terms: int, stream=None):
    """mw_gemm_split_bf16_static: the same product with the library's built-in scratch, for callers
    that cannot allocate a scratch buffer.  Only the output tensor is created here (by torch, as
    for every other call of this binding); the C entry point itself allocates nothing."""
    import torch
    M = A.shape[1] if a_mn else A.shape[0]
    K = A.shape[0] if a_mn else A.shape[1]
    N = B.shape[1] if b_mn else B.shape[0]
    D = torch.empty((M, N), dtype=torch.float32, device=A.device)
    _check(lib().mw_gemm_split_bf16_static(_ptr(A), int(a_mn), _ptr(B), int(b_mn), _ptr(D), M, N, K,
                                           int(terms), _stream_handle(stream)),
           "mw_gemm_split_bf16_static")
    return D


# ---- moving a synthetic problem onto the device -------------------------------------------
def to_device(problem, device="cuda"):
    """Returns (params, x, target) as torch tensors in the problem's storage types."""
    import torch
    st = {"f64": torch.float64, "f32": torch.float32, "bf16_f32acc": torch.bfloat16}[problem.prec]
    gt = torch.float64 if problem.prec == "f64" else torch.float32
    params = [torch.from_numpy(np.ascontiguousarray(p)).to(st).to(device).contiguous()
              for p in problem.params]
    x = torch.from_numpy(np.ascontiguousarray(problem.x)).to(st).to(device).contiguous()
    if problem.loss == "xent_mean":
        target = torch.from_numpy(problem.target.astype(np.int32)).to(device)
    else:
        target = torch.from_numpy(np.ascontiguousarray(problem.target)).to(gt).to(device).contiguous()
    return params, x, target


def net_for(problem, backend="auto", resident_inverse=True, inverse_iters=0, warm_inverse=False) -> Net:
    return Net(problem.layers, problem.batch, problem.prec, problem.loss,
               reseed_every=problem.reseed_every, conv_vijp_iters=problem.conv_vijp_iters,
               backend=backend, inverse_iters=inverse_iters, resident_inverse=resident_inverse,
               frag_block=getattr(problem, "frag_block", 0), warm_inverse=warm_inverse)
