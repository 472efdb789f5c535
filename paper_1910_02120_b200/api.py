"""ctypes binding of libist.so: the same calls as include/ist.h, with torch tensors as the
owners of device memory.  Argument marshalling only; every step of a round runs inside the
library's CUDA kernels.  There is no CPU fallback: if the shared library is missing, import
fails with instructions to build it.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("IST_LIB_PATH") or os.path.join(_HERE, "libist.so")

IST_OK = 0
IST_ERR_ARG, IST_ERR_STATE, IST_ERR_WORKSPACE, IST_ERR_CUDA = -1, -2, -3, -4
IST_ERR_DEVICE_CHECK, IST_ERR_DEVICE_TIMEOUT, IST_ERR_UNSUPPORTED = -5, -6, -7
IST_FP32, IST_BF16 = 0, 1
IST_X_DENSE_F32, IST_X_DENSE_BF16, IST_X_CSR = 0, 1, 2

EXPORTS = [
    "ist_workspace_bytes", "ist_create", "ist_bind_weights", "ist_partition", "ist_get_partition",
    "ist_get_subnet_params", "ist_local_steps", "ist_reassemble", "ist_eval", "ist_sync_status",
    "ist_kernel_launches", "ist_last_error", "ist_destroy", "ist_profile", "ist_profile_read",
    "ist_partition_layer_static", "ist_norm_workspace_bytes", "ist_enable_normalization", "ist_calibrate",
    "ist_set_subnet_range", "ist_packed_layer", "ist_workspace_bytes2", "ist_create2",
    "ist_selftest_wait_expiry", "ist_subnet_slice_shape", "ist_static_partition_status", "ist_local_steps_dx",
]
IST_PART_BALANCED, IST_PART_IID = 0, 1
IST_STATIC_MAX_NEURONS, IST_STATIC_MAX_SUBNETS = 65536, 64

KERNEL_CLASSES = ["partition", "gather", "stage", "fwd", "loss", "dx", "dw_sgd", "bias_sgd", "spmm",
                  "scatter", "eval", "norm"]


class IstInput(ctypes.Structure):
    _fields_ = [
        ("kind", ctypes.c_int32),
        ("batch", ctypes.c_int32),
        ("dense", ctypes.c_void_p),
        ("row_ptr", ctypes.c_void_p),
        ("col", ctypes.c_void_p),
        ("val", ctypes.c_void_p),
        ("stride_subnet", ctypes.c_int64),
        ("stride_step", ctypes.c_int64),
    ]


class IstError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"ist_status {status}: {message}")
        self.status = status


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_1910_02120_b200.build` "
            "(needs nvcc); there is no fallback implementation")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, u64, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_uint64, ctypes.c_size_t
    p64 = ctypes.POINTER(ctypes.c_int64)
    lib.ist_workspace_bytes.restype = sz
    lib.ist_workspace_bytes.argtypes = [p64, i32, i32, i32, i32, i32]
    lib.ist_workspace_bytes2.restype = sz
    lib.ist_workspace_bytes2.argtypes = [p64, i32, i32, i32, i32, i32, i32]
    lib.ist_create2.restype = ctypes.c_int32
    lib.ist_create2.argtypes = [ctypes.POINTER(vp), p64, i32, i32, i32, i32, i32, i32, vp, sz, vp]
    lib.ist_create.restype = ctypes.c_int32
    lib.ist_create.argtypes = [ctypes.POINTER(vp), p64, i32, i32, i32, i32, i32, vp, sz, vp]
    lib.ist_bind_weights.restype = ctypes.c_int32
    lib.ist_bind_weights.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp)]
    lib.ist_partition.restype = ctypes.c_int32
    lib.ist_partition.argtypes = [vp, u64]
    lib.ist_get_partition.restype = ctypes.c_int32
    lib.ist_get_partition.argtypes = [vp, i32, vp, vp]
    lib.ist_get_subnet_params.restype = ctypes.c_int32
    lib.ist_get_subnet_params.argtypes = [vp, i32, i32, vp, vp]
    lib.ist_subnet_slice_shape.restype = ctypes.c_int32
    lib.ist_subnet_slice_shape.argtypes = [vp, i32, i32, p64, p64]
    lib.ist_static_partition_status.restype = ctypes.c_int32
    lib.ist_static_partition_status.argtypes = [vp]
    lib.ist_local_steps.restype = ctypes.c_int32
    lib.ist_local_steps.argtypes = [vp, ctypes.POINTER(IstInput), vp, ctypes.c_float, i32, vp]
    lib.ist_local_steps_dx.restype = ctypes.c_int32
    lib.ist_local_steps_dx.argtypes = [vp, ctypes.POINTER(IstInput), vp, ctypes.c_float, i32, vp, vp]
    lib.ist_reassemble.restype = ctypes.c_int32
    lib.ist_reassemble.argtypes = [vp]
    lib.ist_eval.restype = ctypes.c_int32
    lib.ist_eval.argtypes = [vp, ctypes.POINTER(IstInput), vp, i64, vp, vp]
    lib.ist_sync_status.restype = ctypes.c_int32
    lib.ist_sync_status.argtypes = [vp]
    lib.ist_selftest_wait_expiry.restype = ctypes.c_int32
    lib.ist_selftest_wait_expiry.argtypes = [vp, i64]
    lib.ist_kernel_launches.restype = i64
    lib.ist_kernel_launches.argtypes = [vp]
    lib.ist_last_error.restype = ctypes.c_char_p
    lib.ist_last_error.argtypes = [vp]
    lib.ist_profile.restype = ctypes.c_int32
    lib.ist_profile.argtypes = [vp, i32]
    lib.ist_profile_read.restype = ctypes.c_int32
    lib.ist_profile_read.argtypes = [vp, i32, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_double)]
    lib.ist_partition_layer_static.restype = ctypes.c_int32
    lib.ist_partition_layer_static.argtypes = [u64, i32, i64, i32, vp, vp, vp]
    lib.ist_destroy.restype = None
    lib.ist_norm_workspace_bytes.argtypes = [vp]
    lib.ist_norm_workspace_bytes.restype = sz
    lib.ist_enable_normalization.argtypes = [vp, ctypes.c_float, vp, sz]
    lib.ist_enable_normalization.restype = i32
    lib.ist_calibrate.argtypes = [vp, ctypes.POINTER(IstInput), i64]
    lib.ist_calibrate.restype = i32
    lib.ist_set_subnet_range.argtypes = [vp, i32, i32]
    lib.ist_set_subnet_range.restype = i32
    lib.ist_packed_layer.argtypes = [vp, i32, ctypes.POINTER(vp), ctypes.POINTER(sz), ctypes.POINTER(vp),
                                     ctypes.POINTER(sz)]
    lib.ist_packed_layer.restype = i32
    lib.ist_destroy.argtypes = [vp]
    return lib


lib = _load()


def _dims(layer_dims: Sequence[int]):
    arr = (ctypes.c_int64 * len(layer_dims))(*[int(d) for d in layer_dims])
    return arr, len(layer_dims)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _check(handle, status: int):
    if status != IST_OK:
        raise IstError(status, lib.ist_last_error(handle).decode())


def ist_workspace_bytes2(layer_dims, S, precision, max_batch, input_is_csr=False, partition_rule=0) -> int:
    arr, n = _dims(layer_dims)
    return int(lib.ist_workspace_bytes2(arr, n, S, precision, max_batch, int(bool(input_is_csr)), partition_rule))


def ist_workspace_bytes(layer_dims, S, precision, max_batch, input_is_csr=False) -> int:
    arr, n = _dims(layer_dims)
    return int(lib.ist_workspace_bytes(arr, n, S, precision, max_batch, int(bool(input_is_csr))))


def make_input(X, batch: int, stride_subnet: int, stride_step: int) -> Tuple[IstInput, tuple]:
    """X: a CUDA tensor of rows (fp32 or bf16, last dim N_0) or a (row_ptr, col, val) triple of
    CUDA tensors (int32, int32, fp32).  Returns the struct and the tensors it points into."""
    inp = IstInput()
    inp.batch = int(batch)
    inp.stride_subnet = int(stride_subnet)
    inp.stride_step = int(stride_step)
    if isinstance(X, (tuple, list)):
        rp, col, val = X
        assert rp.dtype == torch.int32 and col.dtype == torch.int32 and val.dtype == torch.float32
        assert rp.is_cuda and col.is_cuda and val.is_cuda
        inp.kind = IST_X_CSR
        inp.row_ptr, inp.col, inp.val = rp.data_ptr(), col.data_ptr(), val.data_ptr()
        return inp, (rp, col, val)
    assert X.is_cuda and X.is_contiguous()
    if X.dtype == torch.float32:
        inp.kind = IST_X_DENSE_F32
    elif X.dtype == torch.bfloat16:
        inp.kind = IST_X_DENSE_BF16
    else:
        raise TypeError(f"unsupported input dtype {X.dtype}")
    inp.dense = X.data_ptr()
    return inp, (X,)


def ist_partition_layer_static(seed: int, hidden_layer: int, n_neurons: int, S: int,
                               idx_out: torch.Tensor, off_out: torch.Tensor,
                               stream: Optional[torch.cuda.Stream] = None) -> int:
    """Partition of one hidden layer into caller-owned int32 tensors, using the library's built-in
    device scratch instead of a workspace (for callers that must not allocate).  Returns the
    ist_status; work is asynchronous on `stream` (default: the current stream of idx_out's device)."""
    assert idx_out.is_cuda and idx_out.dtype == torch.int32 and idx_out.numel() >= n_neurons
    assert off_out.is_cuda and off_out.dtype == torch.int32 and off_out.numel() >= S + 1
    with torch.cuda.device(idx_out.device):
        s = stream if stream is not None else torch.cuda.current_stream(idx_out.device)
        return int(lib.ist_partition_layer_static(ctypes.c_uint64(seed & (2 ** 64 - 1)), hidden_layer, n_neurons, S,
                                                  idx_out.data_ptr(), off_out.data_ptr(),
                                                  ctypes.c_void_p(s.cuda_stream)))


def ist_static_partition_status(stream: Optional[torch.cuda.Stream] = None, device=None) -> int:
    """Waits for `stream` and returns the device status word of ist_partition_layer_static's kernels
    on the current device (IST_OK unless one of their bounds checks tripped)."""
    dev = torch.device(device) if device is not None else torch.device("cuda", torch.cuda.current_device())
    with torch.cuda.device(dev):
        s = stream if stream is not None else torch.cuda.current_stream(dev)
        return int(lib.ist_static_partition_status(ctypes.c_void_p(s.cuda_stream)))


class Ist:
    """One IST context: owns the workspace tensor, borrows the full network's tensors.

    Method names mirror the C calls (ist_partition -> partition, ...)."""

    def __init__(self, layer_dims: Sequence[int], S: int, precision: int, max_batch: int,
                 input_is_csr: bool = False, device: str = "cuda:0", stream: Optional[torch.cuda.Stream] = None,
                 partition_rule: int = IST_PART_BALANCED):
        self.partition_rule = int(partition_rule)
        self.layer_dims = [int(d) for d in layer_dims]
        self.t = len(self.layer_dims) - 1
        self.S, self.precision, self.max_batch = int(S), int(precision), int(max_batch)
        self.input_is_csr = bool(input_is_csr)
        self.device = torch.device(device)
        self.stream = stream
        self.handle = ctypes.c_void_p()
        nbytes = ist_workspace_bytes2(self.layer_dims, S, precision, max_batch, input_is_csr, self.partition_rule)
        if nbytes == 0:
            raise IstError(IST_ERR_ARG, lib.ist_last_error(None).decode())
        self.workspace_bytes = nbytes
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            arr, n = _dims(self.layer_dims)
            st = lib.ist_create2(ctypes.byref(self.handle), arr, n, self.S, self.precision, self.max_batch,
                                 int(self.input_is_csr), self.partition_rule, self.workspace.data_ptr(), nbytes,
                                 self._stream_ptr())
        if st != IST_OK:
            self.handle = ctypes.c_void_p()
            raise IstError(st, lib.ist_last_error(None).decode())
        self.W: List[torch.Tensor] = []
        self.b: List[torch.Tensor] = []

    def _stream_ptr(self):
        s = self.stream if self.stream is not None else torch.cuda.current_stream(self.device)
        return ctypes.c_void_p(s.cuda_stream)

    def close(self):
        if getattr(self, "handle", None) and self.handle.value:
            lib.ist_destroy(self.handle)
            self.handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # --- calls -----------------------------------------------------------------------------
    def bind_weights(self, W: Sequence[torch.Tensor], b: Sequence[torch.Tensor]):
        assert len(W) == self.t and len(b) == self.t
        for l in range(self.t):
            assert W[l].is_cuda and W[l].dtype == torch.float32 and W[l].is_contiguous()
            assert tuple(W[l].shape) == (self.layer_dims[l], self.layer_dims[l + 1])
            assert b[l].is_cuda and b[l].dtype == torch.float32 and tuple(b[l].shape) == (self.layer_dims[l + 1],)
        self.W, self.b = list(W), list(b)
        Wp = (ctypes.c_void_p * self.t)(*[w.data_ptr() for w in W])
        bp = (ctypes.c_void_p * self.t)(*[v.data_ptr() for v in b])
        _check(self.handle, lib.ist_bind_weights(self.handle, Wp, bp))

    def partition(self, seed: int):
        _check(self.handle, lib.ist_partition(self.handle, ctypes.c_uint64(seed & (2 ** 64 - 1))))

    def get_partition(self, hidden_layer: int):
        idx = torch.empty(self.layer_dims[hidden_layer], dtype=torch.int32, device=self.device)
        off = torch.empty(self.S + 1, dtype=torch.int32, device=self.device)
        _check(self.handle, lib.ist_get_partition(self.handle, hidden_layer, idx.data_ptr(), off.data_ptr()))
        return idx, off

    def subnet_slice_shape(self, layer: int, s: int) -> Tuple[int, int]:
        """(rows, cols) of subnet s's slice of layer `layer` under the partition in place."""
        rows, cols = ctypes.c_int64(), ctypes.c_int64()
        _check(self.handle, lib.ist_subnet_slice_shape(self.handle, layer, s, ctypes.byref(rows), ctypes.byref(cols)))
        return int(rows.value), int(cols.value)

    def get_subnet_params(self, layer: int, s: int):
        rows, cols = self.subnet_slice_shape(layer, s)
        Wt = torch.empty((rows, cols), dtype=torch.float32, device=self.device)
        bt = torch.empty(cols, dtype=torch.float32, device=self.device)
        _check(self.handle, lib.ist_get_subnet_params(self.handle, layer, s, Wt.data_ptr(), bt.data_ptr()))
        return Wt, bt

    def local_steps(self, X, y: torch.Tensor, lr: float, K: int, batch: int,
                    stride_subnet: Optional[int] = None, stride_step: Optional[int] = None,
                    loss_out: Optional[torch.Tensor] = None, want_loss: bool = True,
                    dx_out: Optional[torch.Tensor] = None):
        """X rows ordered [S][K][batch] by default (stride_subnet = K*batch, stride_step = batch).
        dx_out: fp32 [rows of X][N_0], receives the loss gradient with respect to every input row
        (ist_local_steps_dx)."""
        if stride_subnet is None:
            stride_subnet = K * batch
        if stride_step is None:
            stride_step = batch
        inp, keep = make_input(X, batch, stride_subnet, stride_step)
        assert y.is_cuda and y.dtype == torch.int32 and y.is_contiguous()
        n_sub = getattr(self, "sub_count", self.S)
        if loss_out is None and want_loss:
            loss_out = torch.empty(n_sub * K, dtype=torch.float32, device=self.device)
        if dx_out is not None:
            assert dx_out.is_cuda and dx_out.dtype == torch.float32 and dx_out.is_contiguous()
            _check(self.handle, lib.ist_local_steps_dx(self.handle, ctypes.byref(inp), y.data_ptr(),
                                                       ctypes.c_float(lr), K, _ptr(loss_out), dx_out.data_ptr()))
        else:
            _check(self.handle, lib.ist_local_steps(self.handle, ctypes.byref(inp), y.data_ptr(),
                                                    ctypes.c_float(lr), K, _ptr(loss_out)))
        return loss_out.view(n_sub, K) if loss_out is not None else None

    def reassemble(self):
        _check(self.handle, lib.ist_reassemble(self.handle))

    def eval(self, X, y: torch.Tensor, n: int):
        inp, keep = make_input(X, 0, 0, 0)
        loss = torch.empty(1, dtype=torch.float32, device=self.device)
        correct = torch.empty(1, dtype=torch.int64, device=self.device)
        _check(self.handle, lib.ist_eval(self.handle, ctypes.byref(inp), y.data_ptr(), n,
                                         loss.data_ptr(), correct.data_ptr()))
        return loss, correct

    def set_subnet_range(self, first: int, count: int):
        """Train only subnets first .. first+count-1 in local_steps (the others are trained elsewhere)."""
        _check(self.handle, lib.ist_set_subnet_range(self.handle, first, count))
        self.sub_first, self.sub_count = first, count

    def packed_layer(self, layer: int):
        """(master [S][elems] fp32, bias [S][ld] fp32): views of the workspace, for the slice exchange."""
        mp, mb, bp, bb = ctypes.c_void_p(), ctypes.c_size_t(), ctypes.c_void_p(), ctypes.c_size_t()
        _check(self.handle, lib.ist_packed_layer(self.handle, layer, ctypes.byref(mp), ctypes.byref(mb),
                                                 ctypes.byref(bp), ctypes.byref(bb)))
        base = self.workspace.data_ptr()

        def view(ptr, nbytes):
            off = ptr.value - base
            return self.workspace[off:off + self.S * nbytes].view(torch.float32).view(self.S, nbytes // 4)

        return view(mp, mb.value), view(bp, bb.value)

    def enable_normalization(self, eps: float):
        """Sec. 2.2 batch standardisation of the hidden layers for all later calls."""
        nbytes = int(lib.ist_norm_workspace_bytes(self.handle))
        with torch.cuda.device(self.device):
            self.norm_workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        _check(self.handle, lib.ist_enable_normalization(self.handle, ctypes.c_float(eps),
                                                         self.norm_workspace.data_ptr(), nbytes))

    def calibrate(self, X, n: int):
        inp, keep = make_input(X, 0, 0, 0)
        _check(self.handle, lib.ist_calibrate(self.handle, ctypes.byref(inp), n))

    def sync_status(self):
        _check(self.handle, lib.ist_sync_status(self.handle))

    def selftest_wait_expiry(self, limit_cycles: int):
        """Enqueues a kernel whose bounded wait must expire; sync_status() then raises with
        IST_ERR_DEVICE_TIMEOUT."""
        _check(self.handle, lib.ist_selftest_wait_expiry(self.handle, int(limit_cycles)))

    def profile(self, enable: bool):
        _check(self.handle, lib.ist_profile(self.handle, int(bool(enable))))

    def profile_read(self):
        """{class name: (kernels launched, device milliseconds)} since profiling was enabled."""
        out = {}
        for k, name in enumerate(KERNEL_CLASSES):
            n, ms = ctypes.c_int64(), ctypes.c_double()
            _check(self.handle, lib.ist_profile_read(self.handle, k, ctypes.byref(n), ctypes.byref(ms)))
            out[name] = (int(n.value), float(ms.value))
        return out

    def kernel_launches(self) -> int:
        return int(lib.ist_kernel_launches(self.handle))

    # --- one whole round ---------------------------------------------------------------------
    def round(self, seed: int, X, y, lr: float, K: int, batch: int, loss_out=None, want_loss=True):
        self.partition(seed)
        loss = self.local_steps(X, y, lr, K, batch, loss_out=loss_out, want_loss=want_loss)
        self.reassemble()
        return loss
