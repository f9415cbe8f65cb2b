"""ctypes binding of libtm.so: same entry points as include/tm.h, tensors in, tensors out.

Argument marshalling only.  torch is used for device memory and streams."""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

TM_EXACT, TM_APPROX, TM_APPROX_COVER = 0, 1, 2
TM_F32, TM_BF16 = 0, 1
TM_DEV_NONFINITE, TM_DEV_INTERNAL, TM_DEV_BADMASK = 1, 2, 4
TM_NM1D_ABSORB_MEAN = 1
TM_ERR_TOO_LARGE, TM_ERR_CAPTURE = 9, 10

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libtm.so")
_lib = None


class TmError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__("tm error %d: %s" % (code, what))
        self.code = code


class tm_problem(ctypes.Structure):
    _fields_ = [("W", ctypes.c_void_p), ("rows", ctypes.c_int64), ("cols", ctypes.c_int64), ("ld", ctypes.c_int64),
                ("dtype", ctypes.c_int32), ("mask_out", ctypes.c_void_p), ("masked_w_out", ctypes.c_void_p),
                ("objective_out", ctypes.c_void_p)]


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Loads libtm.so (built in-tree by ``python -m paper_2102_08124_b200.build``).  Raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise TmError(-1, "libtm.so is not built; run `python -m paper_2102_08124_b200.build` (there is no CPU fallback)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
    lib.tm_mask_words_per_row.argtypes = [i64]; lib.tm_mask_words_per_row.restype = sz
    lib.tm_mask_words.argtypes = [i64, i64]; lib.tm_mask_words.restype = sz
    for f in (lib.tm_find_mask, lib.tm_find_mask_bf16):
        f.argtypes = [vp, i64, i64, i32, i32, i32, vp, vp, vp]; f.restype = i32
    lib.tm_device_status.argtypes = [ctypes.POINTER(i32)]; lib.tm_device_status.restype = i32
    lib.tm_find_mask_batched.argtypes = [ctypes.POINTER(tm_problem), i32, i32, i32, i32, vp, sz, vp, vp]
    lib.tm_find_mask_batched.restype = i32
    lib.tm_find_mask_batched_static.argtypes = [ctypes.POINTER(tm_problem), i32, i32, i32, i32, vp, vp]
    lib.tm_find_mask_batched_static.restype = i32
    lib.tm_workspace_bytes.argtypes = [ctypes.POINTER(tm_problem), i32]; lib.tm_workspace_bytes.restype = sz
    lib.tm_find_mask_host.argtypes = [vp, i32, i64, i64, i32, i32, i32, vp, vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i32)]
    lib.tm_find_mask_host.restype = i32
    lib.tm_plan_create.argtypes = [ctypes.POINTER(tm_problem), i32, i32, i32, i32, vp, sz, ctypes.POINTER(vp)]; lib.tm_plan_create.restype = i32
    lib.tm_plan_run.argtypes = [vp, vp, vp]; lib.tm_plan_run.restype = i32
    lib.tm_plan_destroy.argtypes = [vp]; lib.tm_plan_destroy.restype = None
    u64p = ctypes.c_void_p
    lib.tm_aux_workspace_bytes.restype = sz
    lib.tm_nm_mask_1d.argtypes = [ctypes.POINTER(tm_problem), i32, i32, i32, u64p, vp, sz, vp, vp]; lib.tm_nm_mask_1d.restype = i32
    lib.tm_mask_violations.argtypes = [vp, i32, i64, i64, i64, vp, u64p, vp, sz, vp]; lib.tm_mask_violations.restype = i32
    lib.tm_compress_2_4.argtypes = [vp, i32, i64, i64, i64, vp, vp, vp, vp, vp, vp, vp]; lib.tm_compress_2_4.restype = i32
    lib.tm_mask_hamming.argtypes = [vp, vp, i64, u64p, vp, sz, vp]; lib.tm_mask_hamming.restype = i32
    lib.tm_status_string.argtypes = [i32]; lib.tm_status_string.restype = ctypes.c_char_p
    lib.tm_version.restype = i32
    _lib = lib
    return lib


def tm_status_string(code: int) -> str:
    return load_library().tm_status_string(code).decode()


def tm_version() -> int:
    return int(load_library().tm_version())


def tm_mask_words_per_row(cols: int) -> int:
    return int(load_library().tm_mask_words_per_row(cols))


def tm_mask_words(rows: int, cols: int) -> int:
    return int(load_library().tm_mask_words(rows, cols))


def _check(rc: int):
    if rc != 0:
        raise TmError(rc, tm_status_string(rc))


def _dtype_code(t) -> int:
    import torch
    if t.dtype == torch.float32:
        return TM_F32
    if t.dtype == torch.bfloat16:
        return TM_BF16
    raise TmError(5, "W must be float32 or bfloat16")


def _outputs(W, mask_out, masked_w_out, objective_out, want_masked, want_objective):
    import torch
    rows, cols = W.shape
    if mask_out is None:
        mask_out = torch.empty((rows, tm_mask_words_per_row(cols)), dtype=torch.int32, device=W.device)
    if masked_w_out is None and want_masked:
        masked_w_out = torch.empty_like(W)
    if objective_out is None and want_objective:
        objective_out = torch.empty((1,), dtype=torch.float64, device=W.device)
    return mask_out, masked_w_out, objective_out


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _plain(fn_name, W, N, M, method, mask_out, masked_w_out, objective_out, want_masked, want_objective):
    import torch
    lib = load_library()
    if not (W.is_cuda and W.dim() == 2 and W.is_contiguous()):
        raise TmError(2, "W must be a contiguous 2-D CUDA tensor")
    mask_out, masked_w_out, objective_out = _outputs(W, mask_out, masked_w_out, objective_out, want_masked, want_objective)
    with torch.cuda.device(W.device):
        _check(getattr(lib, fn_name)(_ptr(W), W.shape[0], W.shape[1], N, M, method, _ptr(mask_out), _ptr(masked_w_out), _ptr(objective_out)))
    return mask_out, masked_w_out, objective_out


def tm_find_mask(W, N: int, M: int, method: int, mask_out=None, masked_w_out=None, objective_out=None,
                 want_masked: bool = True, want_objective: bool = True):
    """fp32 matrix on the legacy default stream.  Returns (mask int32[rows, wpr], masked W or None, objective[1] or None)."""
    import torch
    if W.dtype != torch.float32:
        raise TmError(5, "tm_find_mask takes float32; use tm_find_mask_bf16 for bfloat16")
    return _plain("tm_find_mask", W, N, M, method, mask_out, masked_w_out, objective_out, want_masked, want_objective)


def tm_find_mask_bf16(W, N: int, M: int, method: int, mask_out=None, masked_w_out=None, objective_out=None,
                      want_masked: bool = True, want_objective: bool = True):
    import torch
    if W.dtype != torch.bfloat16:
        raise TmError(5, "tm_find_mask_bf16 takes bfloat16")
    return _plain("tm_find_mask_bf16", W, N, M, method, mask_out, masked_w_out, objective_out, want_masked, want_objective)


def tm_device_status() -> int:
    s = ctypes.c_int(0)
    _check(load_library().tm_device_status(ctypes.byref(s)))
    return s.value


def _problem_array(Ws: Sequence, masks, maskeds, objectives):
    arr = (tm_problem * max(len(Ws), 1))()
    for k, W in enumerate(Ws):
        arr[k].W = W.data_ptr(); arr[k].rows = W.shape[0]; arr[k].cols = W.shape[1]; arr[k].ld = W.stride(0) if W.shape[0] > 1 else W.shape[1]
        arr[k].dtype = _dtype_code(W)
        arr[k].mask_out = masks[k].data_ptr()
        arr[k].masked_w_out = maskeds[k].data_ptr() if maskeds is not None and maskeds[k] is not None else None
        arr[k].objective_out = objectives[k:k + 1].data_ptr() if objectives is not None else None
    return arr


def _batch_outputs(Ws: Sequence, masks, maskeds, objectives, workspace, status, want_masked: bool):
    """Checks the matrices of a batched call and creates whichever output tensors the caller did not pass."""
    import torch
    dev = Ws[0].device
    for W in Ws:
        if not (W.is_cuda and W.dim() == 2 and (W.shape[1] <= 1 or W.stride(1) == 1) and W.device == dev):
            raise TmError(2, "every W must be a 2-D CUDA tensor with unit column stride on one device")
    if masks is None:
        masks = [torch.empty((W.shape[0], tm_mask_words_per_row(W.shape[1])), dtype=torch.int32, device=dev) for W in Ws]
    if maskeds is None and want_masked:
        maskeds = [torch.empty_strided(W.shape, W.stride(), dtype=W.dtype, device=dev) for W in Ws]
    if maskeds is not None:
        for W, Y in zip(Ws, maskeds):                      # the ABI has one leading dimension per matrix
            if Y is not None and (Y.shape != W.shape or Y.stride() != W.stride() or Y.dtype != W.dtype):
                raise TmError(2, "masked_w_out must have the shape, strides and dtype of W")
    if objectives is None:
        objectives = torch.empty((len(Ws),), dtype=torch.float64, device=dev)
    if status is None:
        status = torch.zeros((1,), dtype=torch.int32, device=dev)
    if workspace is None:
        workspace = torch.empty((tm_workspace_bytes(len(Ws)),), dtype=torch.uint8, device=dev)
    return dev, masks, maskeds, objectives, status, workspace


class TmBatch:
    """A list of matrices with their output tensors, marshalled once into the C descriptor array.

    Filling the descriptors costs a few microseconds per matrix in Python; a training loop that re-derives the
    masks of the same weight buffers every few iterations prepares the batch once and calls run() each time."""

    def __init__(self, Ws: Sequence, masks=None, maskeds=None, objectives=None, workspace=None, status=None, want_masked: bool = True):
        if len(Ws) == 0:
            raise TmError(2, "empty batch")
        dev, masks, maskeds, objectives, status, workspace = _batch_outputs(Ws, masks, maskeds, objectives, workspace, status, want_masked)
        self.Ws, self.masks, self.maskeds, self.objectives, self.status, self.workspace = list(Ws), masks, maskeds, objectives, status, workspace
        self.device = dev
        self.count = len(Ws)
        self._arr = _problem_array(Ws, masks, maskeds, objectives)
        self._lib = load_library()

    def run(self, N: int, M: int, method: int, stream=None):
        """tm_find_mask_batched on the prepared descriptors; asynchronous on `stream` or torch's current stream."""
        import torch
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        with torch.cuda.device(self.device):
            _check(self._lib.tm_find_mask_batched(self._arr, self.count, N, M, method, _ptr(self.workspace), self.workspace.numel(),
                                                  _ptr(self.status), ctypes.c_void_p(s.cuda_stream)))
        return self.masks, self.maskeds, self.objectives, self.status


class TmPlan:
    """Handle of a prepared batched search (see tm_plan_create in include/tm.h); owns its tensors."""

    def __init__(self, handle, batch, N, M, method):
        self._handle, self.batch, self.N, self.M, self.method = handle, batch, N, M, method

    def __del__(self):
        try:
            tm_plan_destroy(self)
        except Exception:
            pass


def tm_plan_create(Ws: Sequence, N: int, M: int, method: int, masks=None, maskeds=None, objectives=None, workspace=None,
                   status=None, want_masked: bool = True) -> TmPlan:
    """Validates and prepares a batched search once: descriptors, tensor maps and device tables.  tm_plan_run() then
    only launches kernels (it can be captured into a CUDA graph)."""
    import torch
    batch = TmBatch(Ws, masks, maskeds, objectives, workspace, status, want_masked)
    h = ctypes.c_void_p()
    with torch.cuda.device(batch.device):
        _check(batch._lib.tm_plan_create(batch._arr, batch.count, N, M, method, _ptr(batch.workspace), batch.workspace.numel(), ctypes.byref(h)))
    return TmPlan(h, batch, N, M, method)


def tm_plan_run(plan: TmPlan, status=None, stream=None):
    """Launches the prepared search on `stream` (or torch's current stream).  Returns (masks, maskeds, objectives, status)."""
    import torch
    b = plan.batch
    st = status if status is not None else b.status
    with torch.cuda.device(b.device):
        _check(b._lib.tm_plan_run(plan._handle, _ptr(st), _stream_ptr(b.device, stream)))
    return b.masks, b.maskeds, b.objectives, st


def tm_plan_destroy(plan: TmPlan):
    if plan._handle is not None and plan._handle.value:
        plan.batch._lib.tm_plan_destroy(plan._handle)
        plan._handle = None


def tm_workspace_bytes(count: int) -> int:
    return int(load_library().tm_workspace_bytes(None, count))


def tm_find_mask_batched(Ws: Sequence, N: int, M: int, method: int, masks=None, maskeds=None, objectives=None,
                         workspace=None, status=None, stream=None, want_masked: bool = True):
    """One launch for a list of 2-D CUDA tensors (fp32 and/or bf16; rows may be strided, stride(1) == 1).

    Returns (masks, maskeds, objectives float64[count], status int32[1], workspace uint8[...]).  Runs on
    `stream` (a torch.cuda.Stream) or on torch's current stream.  With more than one matrix the descriptor tables
    are copied from host memory first (the runtime may wait for the stream's earlier work to do so), and such a
    call is refused on a capturing stream: capture tm_plan_run() instead."""
    import torch
    lib = load_library()
    if len(Ws) == 0:
        return [], [], None, status, workspace
    dev, masks, maskeds, objectives, status, workspace = _batch_outputs(Ws, masks, maskeds, objectives, workspace, status, want_masked)
    arr = _problem_array(Ws, masks, maskeds, objectives)
    with torch.cuda.device(dev):
        s = stream if stream is not None else torch.cuda.current_stream(dev)
        _check(lib.tm_find_mask_batched(arr, len(Ws), N, M, method, _ptr(workspace), workspace.numel(), _ptr(status),
                                        ctypes.c_void_p(s.cuda_stream)))
    return masks, maskeds, objectives, status, workspace


TM_STATIC_MAX_MATRICES = 16


def tm_find_mask_batched_static(Ws: Sequence, N: int, M: int, method: int, masks, maskeds, objectives, status, stream=None):
    """tm_find_mask_batched() for callers that must not allocate device memory (a plug-in inside another
    framework's memory pool, a pre-allocated real-time loop): the library's built-in scratch replaces the
    workspace, at most TM_STATIC_MAX_MATRICES matrices per call.  Every output tensor is passed in (masks:
    list of int32 [rows, wpr]; maskeds: list of tensors shaped like W, or None; objectives: float64[count];
    status: int32[1]); this function creates no tensor.  The caller must order the calls on a device: calls that
    overlap on the GPU share the scratch, which for more than one matrix also holds the descriptor tables and
    tensor maps, so an unordered second call can redirect the loads and stores of a running one (wrong outputs,
    out-of-range accesses).  Only single-matrix calls confine such a race to the objective value."""
    import torch
    lib = load_library()
    dev = Ws[0].device if len(Ws) else torch.device("cuda")
    arr = _problem_array(Ws, masks, maskeds, objectives)
    with torch.cuda.device(dev):
        s = stream if stream is not None else torch.cuda.current_stream(dev)
        _check(lib.tm_find_mask_batched_static(arr, len(Ws), N, M, method, _ptr(status), ctypes.c_void_p(s.cuda_stream)))


def tm_aux_workspace_bytes() -> int:
    return int(load_library().tm_aux_workspace_bytes())


def _aux_workspace(dev, workspace):
    import torch
    if workspace is None:
        workspace = torch.empty((tm_aux_workspace_bytes(),), dtype=torch.uint8, device=dev)
    return workspace


def _stream_ptr(dev, stream):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream(dev)
    return ctypes.c_void_p(s.cuda_stream)


def tm_nm_mask_1d(W, N: int, M: int, absorb_mean: bool = False, mask_out=None, masked_w_out=None, objective_out=None,
                  violations_out=None, status=None, workspace=None, stream=None, want_masked: bool = True):
    """1-D N:M magnitude pruning along rows (N kept per group of M).  Returns (mask, masked, objective[1],
    violations int64[1], status int32[1]); asynchronous on `stream` or torch's current stream."""
    import torch
    lib = load_library()
    if not (W.is_cuda and W.dim() == 2 and (W.shape[1] <= 1 or W.stride(1) == 1)):
        raise TmError(2, "W must be a 2-D CUDA tensor with unit column stride")
    dev = W.device
    if mask_out is None:
        mask_out = torch.empty((W.shape[0], tm_mask_words_per_row(W.shape[1])), dtype=torch.int32, device=dev)
    if masked_w_out is None and want_masked:
        masked_w_out = torch.empty_strided(W.shape, W.stride(), dtype=W.dtype, device=dev)
    if objective_out is None:
        objective_out = torch.empty((1,), dtype=torch.float64, device=dev)
    if violations_out is None:
        violations_out = torch.zeros((1,), dtype=torch.int64, device=dev)
    if status is None:
        status = torch.zeros((1,), dtype=torch.int32, device=dev)
    workspace = _aux_workspace(dev, workspace)
    arr = _problem_array([W], [mask_out], [masked_w_out] if masked_w_out is not None else None, objective_out)
    with torch.cuda.device(dev):
        _check(lib.tm_nm_mask_1d(arr, N, M, TM_NM1D_ABSORB_MEAN if absorb_mean else 0, _ptr(violations_out), _ptr(workspace), workspace.numel(),
                                 _ptr(status), _stream_ptr(dev, stream)))
    return mask_out, masked_w_out, objective_out, violations_out, status


def tm_mask_violations(W, mask, violations_out=None, workspace=None, stream=None):
    """Non-zero weights whose bit in the packed mask is 0.  Returns int64[1] (device)."""
    import torch
    lib = load_library()
    dev = W.device
    if violations_out is None:
        violations_out = torch.zeros((1,), dtype=torch.int64, device=dev)
    workspace = _aux_workspace(dev, workspace)
    with torch.cuda.device(dev):
        _check(lib.tm_mask_violations(_ptr(W), _dtype_code(W), W.shape[0], W.shape[1], W.stride(0) if W.shape[0] > 1 else W.shape[1], _ptr(mask),
                                      _ptr(violations_out), _ptr(workspace), workspace.numel(), _stream_ptr(dev, stream)))
    return violations_out


def tm_mask_hamming(mask_a, mask_b, distance_out=None, workspace=None, stream=None):
    """Number of differing bits of two packed masks (same shape).  Returns int64[1] (device)."""
    import torch
    lib = load_library()
    dev = mask_a.device
    if mask_a.shape != mask_b.shape or not (mask_a.is_contiguous() and mask_b.is_contiguous()):
        raise TmError(2, "masks must be contiguous and of one shape")
    if distance_out is None:
        distance_out = torch.zeros((1,), dtype=torch.int64, device=dev)
    workspace = _aux_workspace(dev, workspace)
    with torch.cuda.device(dev):
        _check(lib.tm_mask_hamming(_ptr(mask_a), _ptr(mask_b), mask_a.numel(), _ptr(distance_out), _ptr(workspace), workspace.numel(),
                                   _stream_ptr(dev, stream)))
    return distance_out


def tm_compress_2_4(W, mask, values=None, meta=None, values_t=None, meta_t=None, status=None, stream=None):
    """2:4 compressed operands of W and W^T from one transposable mask.  Returns (values [rows, cols/2],
    meta int32 [rows, wpr(cols)], values_t [cols, rows/2], meta_t int32 [cols, wpr(rows)], status int32[1])."""
    import torch
    lib = load_library()
    dev = W.device
    rows, cols = W.shape
    if values is None: values = torch.empty((rows, cols // 2), dtype=W.dtype, device=dev)
    if values_t is None: values_t = torch.empty((cols, rows // 2), dtype=W.dtype, device=dev)
    if meta is None: meta = torch.empty((rows, tm_mask_words_per_row(cols)), dtype=torch.int32, device=dev)
    if meta_t is None: meta_t = torch.empty((cols, tm_mask_words_per_row(rows)), dtype=torch.int32, device=dev)
    if status is None: status = torch.zeros((1,), dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        _check(lib.tm_compress_2_4(_ptr(W), _dtype_code(W), rows, cols, W.stride(0) if rows > 1 else cols, _ptr(mask), _ptr(values), _ptr(meta),
                                   _ptr(values_t), _ptr(meta_t), _ptr(status), _stream_ptr(dev, stream)))
    return values, meta, values_t, meta_t, status


def tm_find_mask_host(W, N: int, M: int, method: int, mask_out=None, masked_w_out=None, want_masked: bool = True,
                      device: Optional[int] = None):
    """Host tensors in, host tensors out (pinned memory lets the copies overlap the kernels).

    W: 2-D contiguous CPU tensor, float32 or bfloat16.  Returns (mask, masked or None, objective float, status int)."""
    import torch
    lib = load_library()
    if W.is_cuda or W.dim() != 2 or not W.is_contiguous():
        raise TmError(2, "W must be a contiguous 2-D CPU tensor")
    rows, cols = W.shape
    if mask_out is None:
        mask_out = torch.empty((rows, tm_mask_words_per_row(cols)), dtype=torch.int32).pin_memory()
    if masked_w_out is None and want_masked:
        masked_w_out = torch.empty_like(W).pin_memory()
    obj = ctypes.c_double(0.0); st = ctypes.c_int(0)
    with torch.cuda.device(device if device is not None else torch.cuda.current_device()):
        _check(lib.tm_find_mask_host(_ptr(W), _dtype_code(W), rows, cols, N, M, method, _ptr(mask_out), _ptr(masked_w_out),
                                     ctypes.byref(obj), ctypes.byref(st)))
    return mask_out, masked_w_out, obj.value, st.value
