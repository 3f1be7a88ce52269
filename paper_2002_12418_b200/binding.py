"""ctypes face of the C-ABI library (``include/mnn_conv.h``): same names, argument
marshalling only.  PyTorch appears only in :class:`ConvLayerRunner`, which uses it
for device memory and the current stream; every step of the path runs in the
library's kernels.  There is no fallback: if the shared library is missing,
loading raises.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmnnconv_b200.so")

MNN_OK, MNN_EINVAL, MNN_EUNSUPPORTED, MNN_EWORKSPACE, MNN_EALIGN, MNN_ECUDA, MNN_ENOTCALIBRATED = 0, -1, -2, -3, -4, -5, -6
ALGO_AUTO, ALGO_WINOGRAD, ALGO_GEMM, ALGO_DIRECT = 0, 1, 2, 3
PREC_TF32, PREC_BF16 = 0, 1
OPERAND_AUTO, OPERAND_TF32, OPERAND_BF16, OPERAND_FP32_REF = 0, 1, 2, 3
POINTS_AUTO, POINTS_PAPER, POINTS_UNIT, POINTS_MIXED = 0, 1, 2, 3
GEMM_LHS_AUTO, GEMM_LHS_PATCHES, GEMM_LHS_X, GEMM_LHS_IMPLICIT = 0, 1, 2, 3
FUSED_AUTO, FUSED_NEVER, FUSED_ONLY = 0, 1, 2
STAGE_WEIGHT, STAGE_INPUT, STAGE_CONTRACT, STAGE_OUTPUT, STAGE_ALL = 1, 2, 4, 8, 15
N_CANDIDATES, N_CONSTS = 16, 16
COST_INADMISSIBLE = 0xFFFFFFFFFFFFFFFF
ALGO_NAMES = {ALGO_WINOGRAD: "winograd", ALGO_GEMM: "gemm", ALGO_DIRECT: "direct"}
OPERAND_NAMES = {OPERAND_TF32: "tf32", OPERAND_BF16: "bf16", OPERAND_FP32_REF: "fp32ref", 0: "-"}

EXPORTED = ["mnn_conv_plan", "mnn_conv_plan_ex", "mnn_conv_plan_rect", "mnn_conv_plan_query", "mnn_conv_set_workspace",
            "mnn_conv_prepare_weights", "mnn_conv_run", "mnn_conv_run_stages", "mnn_conv_device_status",
            "mnn_conv_profile", "mnn_conv_profile_read", "mnn_conv_destroy", "mnn_conv_run_static", "mnn_winograd_matrices", "mnn_accuracy_ppm", "mnn_strassen_rule", "mnn_wait_probe", "mnn_calibrate",
            "mnn_set_calibration", "mnn_get_calibration", "mnn_last_error",
            "mnn_net_plan", "mnn_net_query", "mnn_net_set_workspace", "mnn_net_prepare", "mnn_net_run",
            "mnn_net_device_status", "mnn_net_destroy"]
NET_MAX_LAYERS = 128


class ConvOpts(ctypes.Structure):
    _fields_ = [("groups", ctypes.c_int), ("relu", ctypes.c_int), ("precision", ctypes.c_int),
                ("operand", ctypes.c_int), ("passes", ctypes.c_int), ("force_algo", ctypes.c_int),
                ("force_m", ctypes.c_int), ("points_id", ctypes.c_int), ("chunk_images", ctypes.c_int),
                ("gemm_lhs", ctypes.c_int), ("fused", ctypes.c_int), ("strassen", ctypes.c_int), ("reserved", ctypes.c_int * 4)]


class ConvInfo(ctypes.Structure):
    _fields_ = [("algo", ctypes.c_int), ("m", ctypes.c_int), ("alpha", ctypes.c_int), ("precision", ctypes.c_int),
                ("operand", ctypes.c_int), ("passes", ctypes.c_int), ("points_id", ctypes.c_int),
                ("OH", ctypes.c_int), ("OW", ctypes.c_int), ("groups", ctypes.c_int), ("relu", ctypes.c_int),
                ("chunk_images", ctypes.c_int), ("n_chunks", ctypes.c_int), ("launches_per_run", ctypes.c_int),
                ("cin_pad", ctypes.c_int), ("m_row_stride", ctypes.c_int),
                ("chunk_tiles", ctypes.c_longlong), ("workspace_bytes", ctypes.c_longlong),
                ("u_offset", ctypes.c_longlong), ("u_bytes", ctypes.c_longlong),
                ("v_offset", ctypes.c_longlong), ("v_bytes", ctypes.c_longlong),
                ("m_offset", ctypes.c_longlong), ("m_bytes", ctypes.c_longlong),
                ("predicted_error_ppm", ctypes.c_longlong),
                ("chosen_candidate", ctypes.c_int), ("gemm_lhs", ctypes.c_int),
                ("cost_ps", ctypes.c_ulonglong * N_CANDIDATES),
                ("fused", ctypes.c_int), ("paper_n_hat", ctypes.c_int), ("paper_mul", ctypes.c_ulonglong * 4),
                ("strassen", ctypes.c_int), ("rect", ctypes.c_int)]


class LayerDesc(ctypes.Structure):
    _fields_ = [("Cin", ctypes.c_int), ("Cout", ctypes.c_int), ("k", ctypes.c_int), ("stride", ctypes.c_int),
                ("pad", ctypes.c_int), ("dilation", ctypes.c_int), ("groups", ctypes.c_int), ("relu", ctypes.c_int)]


class NetInfo(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int), ("N", ctypes.c_int), ("H", ctypes.c_int), ("W", ctypes.c_int),
                ("out_C", ctypes.c_int), ("out_H", ctypes.c_int), ("out_W", ctypes.c_int),
                ("launches_per_run", ctypes.c_int),
                ("workspace_bytes", ctypes.c_longlong), ("persistent_bytes", ctypes.c_longlong),
                ("transient_bytes", ctypes.c_longlong), ("activation_bytes", ctypes.c_longlong),
                ("sum_of_layer_workspaces", ctypes.c_longlong),
                ("algo", ctypes.c_int * NET_MAX_LAYERS), ("m", ctypes.c_int * NET_MAX_LAYERS),
                ("operand", ctypes.c_int * NET_MAX_LAYERS), ("passes", ctypes.c_int * NET_MAX_LAYERS),
                ("OH", ctypes.c_int * NET_MAX_LAYERS), ("OW", ctypes.c_int * NET_MAX_LAYERS)]


class MnnError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__("mnn_conv error %d: %s" % (code, message))
        self.code = code


_lib = None


def lib():
    """The loaded library (raises OSError if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise OSError("%s is missing: run `python -m paper_2002_12418_b200.build`" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        i, p, ll = ctypes.c_int, ctypes.c_void_p, ctypes.c_longlong
        L.mnn_conv_plan.argtypes = [i] * 9
        L.mnn_conv_plan.restype = p
        L.mnn_conv_plan_ex.argtypes = [i] * 9 + [ctypes.POINTER(ConvOpts)]
        L.mnn_conv_plan_ex.restype = p
        L.mnn_conv_plan_rect.argtypes = [i] * 9 + [ctypes.POINTER(ConvOpts)]
        L.mnn_conv_plan_rect.restype = p
        L.mnn_conv_plan_query.argtypes = [p, ctypes.POINTER(ConvInfo)]
        L.mnn_conv_plan_query.restype = i
        L.mnn_conv_set_workspace.argtypes = [p, p, ll]
        L.mnn_conv_set_workspace.restype = i
        L.mnn_conv_prepare_weights.argtypes = [p, p, p]
        L.mnn_conv_prepare_weights.restype = i
        L.mnn_conv_run.argtypes = [p, p, p, p, p, p]
        L.mnn_conv_run.restype = i
        L.mnn_conv_run_static.argtypes = [p, p, p, p, p, p]
        L.mnn_conv_run_static.restype = i
        L.mnn_conv_run_stages.argtypes = [p, p, p, p, p, p, ctypes.c_uint]
        L.mnn_conv_run_stages.restype = i
        L.mnn_conv_device_status.argtypes = [p, p, ctypes.POINTER(i)]
        L.mnn_conv_device_status.restype = i
        L.mnn_conv_profile.argtypes = [p, i]
        L.mnn_conv_profile.restype = i
        L.mnn_conv_profile_read.argtypes = [p, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(i)]
        L.mnn_conv_profile_read.restype = i
        L.mnn_conv_destroy.argtypes = [p]
        L.mnn_conv_destroy.restype = None
        L.mnn_winograd_matrices.argtypes = [i, i, i, p, p, p]
        L.mnn_winograd_matrices.restype = i
        L.mnn_accuracy_ppm.argtypes = [i] * 5
        L.mnn_accuracy_ppm.restype = ll
        L.mnn_wait_probe.argtypes = [p, p]
        L.mnn_wait_probe.restype = i
        L.mnn_strassen_rule.argtypes = [ll, ll, ll]
        L.mnn_strassen_rule.restype = i
        L.mnn_calibrate.argtypes = [i, p, ctypes.POINTER(ll)]
        L.mnn_calibrate.restype = i
        L.mnn_set_calibration.argtypes = [ctypes.POINTER(ll)]
        L.mnn_set_calibration.restype = i
        L.mnn_get_calibration.argtypes = [ctypes.POINTER(ll)]
        L.mnn_get_calibration.restype = i
        L.mnn_net_plan.argtypes = [i, i, i, i, ctypes.POINTER(LayerDesc), i]
        L.mnn_net_plan.restype = p
        L.mnn_net_query.argtypes = [p, ctypes.POINTER(NetInfo)]
        L.mnn_net_query.restype = i
        L.mnn_net_set_workspace.argtypes = [p, p, ll]
        L.mnn_net_set_workspace.restype = i
        L.mnn_net_prepare.argtypes = [p, ctypes.POINTER(p), p]
        L.mnn_net_prepare.restype = i
        L.mnn_net_run.argtypes = [p, p, ctypes.POINTER(p), ctypes.POINTER(p), p, p]
        L.mnn_net_run.restype = i
        L.mnn_net_device_status.argtypes = [p, p, ctypes.POINTER(i), ctypes.POINTER(i)]
        L.mnn_net_device_status.restype = i
        L.mnn_net_destroy.argtypes = [p]
        L.mnn_net_destroy.restype = None
        L.mnn_last_error.argtypes = []
        L.mnn_last_error.restype = ctypes.c_char_p
        _lib = L
    return _lib


def mnn_last_error() -> str:
    return (lib().mnn_last_error() or b"").decode()


def _check(rc: int) -> None:
    if rc != MNN_OK:
        raise MnnError(rc, mnn_last_error())


def make_opts(groups=1, relu=0, precision=PREC_TF32, operand=0, passes=0, force_algo=0, force_m=0, points_id=0,
              chunk_images=0, gemm_lhs=0, fused=0, strassen=0) -> ConvOpts:
    o = ConvOpts()
    o.groups, o.relu, o.precision, o.operand, o.passes = groups, int(bool(relu)), precision, operand, passes
    o.force_algo, o.force_m, o.points_id, o.chunk_images = force_algo, force_m, points_id, chunk_images
    o.gemm_lhs = gemm_lhs
    o.fused = fused
    o.strassen = strassen
    return o


def mnn_conv_plan(N, Cin, Cout, H, W, k, stride, pad, dilation):
    h = lib().mnn_conv_plan(N, Cin, Cout, H, W, k, stride, pad, dilation)
    if not h:
        raise MnnError(MNN_EINVAL, mnn_last_error())
    return h


def mnn_conv_plan_ex(N, Cin, Cout, H, W, k, stride, pad, dilation, opts: ConvOpts | None):
    h = lib().mnn_conv_plan_ex(N, Cin, Cout, H, W, k, stride, pad, dilation,
                               ctypes.byref(opts) if opts is not None else None)
    if not h:
        raise MnnError(MNN_EINVAL, mnn_last_error())
    return h


def mnn_conv_plan_rect(N, Cin, Cout, H, W, kh, kw, pad_h, pad_w, opts: ConvOpts | None):
    h = lib().mnn_conv_plan_rect(N, Cin, Cout, H, W, kh, kw, pad_h, pad_w, ctypes.byref(opts) if opts is not None else None)
    if not h:
        raise MnnError(MNN_EINVAL, mnn_last_error())
    return h


def mnn_conv_plan_query(plan) -> ConvInfo:
    info = ConvInfo()
    _check(lib().mnn_conv_plan_query(plan, ctypes.byref(info)))
    return info


def mnn_conv_set_workspace(plan, ptr: int, nbytes: int) -> None:
    _check(lib().mnn_conv_set_workspace(plan, ptr, nbytes))


def mnn_conv_prepare_weights(plan, w_ptr: int, stream: int) -> None:
    _check(lib().mnn_conv_prepare_weights(plan, w_ptr, stream))


def mnn_conv_run(plan, x_ptr: int, w_ptr: int, bias_ptr, y_ptr: int, stream: int) -> None:
    _check(lib().mnn_conv_run(plan, x_ptr, w_ptr, bias_ptr, y_ptr, stream))


STATIC_WORKSPACE_BYTES = 32 << 20


def mnn_conv_run_static(plan, x_ptr: int, w_ptr: int, bias_ptr, y_ptr: int, stream: int) -> None:
    """mnn_conv_run on the library's built-in workspace (no allocation anywhere in the call)."""
    _check(lib().mnn_conv_run_static(plan, x_ptr, w_ptr, bias_ptr, y_ptr, stream))


def mnn_conv_run_stages(plan, x_ptr, w_ptr, bias_ptr, y_ptr, stream: int, stage_mask: int) -> None:
    _check(lib().mnn_conv_run_stages(plan, x_ptr, w_ptr, bias_ptr, y_ptr, stream, stage_mask))


def mnn_conv_device_status(plan, stream: int) -> int:
    code = ctypes.c_int(0)
    _check(lib().mnn_conv_device_status(plan, stream, ctypes.byref(code)))
    return code.value


def mnn_conv_profile(plan, enable: bool) -> None:
    _check(lib().mnn_conv_profile(plan, int(bool(enable))))


def mnn_conv_profile_read(plan):
    """([ms per stage], [launches per stage]) of the last run; stages: weight, input, contraction, output."""
    ms = (ctypes.c_float * 4)()
    n = (ctypes.c_int * 4)()
    _check(lib().mnn_conv_profile_read(plan, ms, n))
    return list(ms), list(n)


def mnn_conv_destroy(plan) -> None:
    lib().mnn_conv_destroy(plan)


def mnn_winograd_matrices(m: int, k: int, points_id: int):
    """(At [m x alpha], G [alpha x k], Bt [alpha x alpha]) as nested lists of fp32 values."""
    alpha = m + k - 1
    At = (ctypes.c_float * (m * alpha))()
    G = (ctypes.c_float * (alpha * k))()
    Bt = (ctypes.c_float * (alpha * alpha))()
    _check(lib().mnn_winograd_matrices(m, k, points_id, At, G, Bt))
    rows = lambda a, r, c: [[a[i * c + j] for j in range(c)] for i in range(r)]
    return rows(At, m, alpha), rows(G, alpha, k), rows(Bt, alpha, alpha)


def mnn_accuracy_ppm(m, k, points_id, operand, passes) -> int:
    v = lib().mnn_accuracy_ppm(m, k, points_id, operand, passes)
    if v < 0:
        raise MnnError(MNN_EINVAL, mnn_last_error())
    return int(v)


def mnn_wait_probe(device_word_ptr: int, stream: int) -> None:
    _check(lib().mnn_wait_probe(device_word_ptr, stream))


def mnn_strassen_rule(m: int, n: int, k: int) -> int:
    return int(lib().mnn_strassen_rule(m, n, k))


def mnn_calibrate(device: int, stream: int) -> list[int]:
    c = (ctypes.c_longlong * N_CONSTS)()
    _check(lib().mnn_calibrate(device, stream, c))
    return list(c)


def mnn_set_calibration(consts) -> None:
    c = (ctypes.c_longlong * N_CONSTS)(*list(consts))
    _check(lib().mnn_set_calibration(c))


def mnn_get_calibration() -> list[int]:
    c = (ctypes.c_longlong * N_CONSTS)()
    _check(lib().mnn_get_calibration(c))
    return list(c)


def mnn_net_plan(N, H, W, layers, precision=PREC_TF32):
    """layers: sequence of objects with Cin, Cout, k, stride, pad, dilation, groups, relu (e.g. workloads.ConvLayer)."""
    arr = (LayerDesc * len(layers))()
    for d, l in zip(arr, layers):
        d.Cin, d.Cout, d.k, d.stride, d.pad, d.dilation = l.Cin, l.Cout, l.k, l.stride, l.pad, l.dilation
        d.groups, d.relu = l.groups, int(bool(l.relu))
    h = lib().mnn_net_plan(N, H, W, len(layers), arr, precision)
    if not h:
        raise MnnError(MNN_EINVAL, mnn_last_error())
    return h


def mnn_net_query(net) -> NetInfo:
    info = NetInfo()
    _check(lib().mnn_net_query(net, ctypes.byref(info)))
    return info


def _ptr_array(ptrs):
    return (ctypes.c_void_p * len(ptrs))(*[ctypes.c_void_p(v) if v else None for v in ptrs])


def mnn_net_set_workspace(net, ptr: int, nbytes: int) -> None:
    _check(lib().mnn_net_set_workspace(net, ptr, nbytes))


def mnn_net_prepare(net, w_ptrs, stream: int) -> None:
    _check(lib().mnn_net_prepare(net, _ptr_array(w_ptrs), stream))


def mnn_net_run(net, x_ptr: int, w_ptrs, bias_ptrs, y_ptr: int, stream: int) -> None:
    _check(lib().mnn_net_run(net, x_ptr, _ptr_array(w_ptrs), _ptr_array(bias_ptrs), y_ptr, stream))


def mnn_net_device_status(net, stream: int):
    code, layer = ctypes.c_int(0), ctypes.c_int(-1)
    _check(lib().mnn_net_device_status(net, stream, ctypes.byref(code), ctypes.byref(layer)))
    return code.value, layer.value


def mnn_net_destroy(net) -> None:
    lib().mnn_net_destroy(net)


class NetRunner:
    """A network plan plus its torch-owned workspace; ``run`` is one mnn_net_run on torch's current stream."""

    def __init__(self, N, H, W, layers, precision=PREC_TF32, device="cuda:0"):
        import torch
        self.torch = torch
        self.device = torch.device(device)
        self.net = mnn_net_plan(N, H, W, layers, precision)
        self.info = mnn_net_query(self.net)
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(self.info.workspace_bytes + 1024, dtype=torch.uint8, device=self.device)
        self._ws_ptr = (self.workspace.data_ptr() + 1023) // 1024 * 1024
        mnn_net_set_workspace(self.net, self._ws_ptr, self.info.workspace_bytes)
        self._keep = None

    def stream(self) -> int:
        return self.torch.cuda.current_stream(self.device).cuda_stream

    def prepare(self, ws) -> None:
        mnn_net_prepare(self.net, [w.data_ptr() for w in ws], self.stream())

    def bind(self, ws, bs) -> None:
        """Marshal the weight / bias pointer arrays once (they are reused by every run)."""
        self._keep = (_ptr_array([w.data_ptr() for w in ws]), _ptr_array([b.data_ptr() if b is not None else 0 for b in bs]))

    def run(self, x, y=None):
        torch = self.torch
        if y is None:
            y = torch.empty((self.info.N, self.info.out_C, self.info.out_H, self.info.out_W), dtype=torch.float32,
                            device=self.device)
        _check(lib().mnn_net_run(self.net, x.data_ptr(), self._keep[0], self._keep[1], y.data_ptr(), self.stream()))
        return y

    def device_status(self):
        return mnn_net_device_status(self.net, self.stream())

    def close(self) -> None:
        if self.net:
            mnn_net_destroy(self.net)
            self.net = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class ConvLayerRunner:
    """A plan plus its torch-owned workspace.  ``run`` launches on torch's current
    stream through mnn_conv_run; nothing here computes."""

    def __init__(self, N, Cin, Cout, H, W, k, stride=1, pad=0, dilation=1, opts: ConvOpts | None = None,
                 device="cuda:0", plan=None):
        import torch
        self.torch = torch
        self.device = torch.device(device)
        self.shape = (N, Cin, Cout, H, W, k, stride, pad, dilation)
        if plan is not None:
            self.plan = plan               # e.g. from mnn_conv_plan_rect; owned by the runner from here on
        else:
            self.plan = mnn_conv_plan_ex(N, Cin, Cout, H, W, k, stride, pad, dilation, opts) if opts is not None \
                else mnn_conv_plan(N, Cin, Cout, H, W, k, stride, pad, dilation)
        self.info = mnn_conv_plan_query(self.plan)
        self.workspace = None
        if self.info.workspace_bytes > 0:
            with torch.cuda.device(self.device):
                self.workspace = torch.empty(self.info.workspace_bytes + 1024, dtype=torch.uint8, device=self.device)
                base = self.workspace.data_ptr()
                self._ws_ptr = (base + 1023) // 1024 * 1024
                mnn_conv_set_workspace(self.plan, self._ws_ptr, self.info.workspace_bytes)

    def stream(self) -> int:
        return self.torch.cuda.current_stream(self.device).cuda_stream

    def prepare(self, w) -> None:
        mnn_conv_prepare_weights(self.plan, w.data_ptr(), self.stream())

    def run(self, x, w, bias=None, y=None, stage_mask=None):
        torch = self.torch
        N, Cin, Cout = self.shape[0], self.shape[1], self.shape[2]
        if y is None:
            y = torch.empty((N, Cout, self.info.OH, self.info.OW), dtype=torch.float32, device=self.device)
        bp = bias.data_ptr() if bias is not None else None
        if stage_mask is None:
            mnn_conv_run(self.plan, x.data_ptr(), w.data_ptr(), bp, y.data_ptr(), self.stream())
        else:
            mnn_conv_run_stages(self.plan, x.data_ptr() if x is not None else None,
                                w.data_ptr() if w is not None else None, bp, y.data_ptr(), self.stream(), stage_mask)
        return y

    def workspace_view(self, offset: int, nbytes: int, dtype):
        """A typed view of a workspace region (for checking the stages one by one)."""
        torch = self.torch
        start = self._ws_ptr - self.workspace.data_ptr() + offset
        return self.workspace[start:start + nbytes].view(dtype)

    def device_status(self) -> int:
        return mnn_conv_device_status(self.plan, self.stream())

    def close(self) -> None:
        if self.plan:
            mnn_conv_destroy(self.plan)
            self.plan = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
