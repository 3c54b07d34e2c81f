"""Handle wrapper: owns a zoa handle, marshals torch tensors to raw pointers.

No arithmetic happens here.  torch supplies device memory for the gradients
and the CUDA stream; the optimizer state lives inside the library.
"""
import numpy as np
import torch

from . import binding as B

_NAMES = {"x": B.BUF_X, "m": B.BUF_M, "u": B.BUF_U, "delta_w": B.BUF_DELTA_W, "v": B.BUF_V,
          "delta_s": B.BUF_DELTA_S, "x_sync": B.BUF_X_SYNC, "words_w": B.BUF_WORDS_W,
          "scales_w": B.BUF_SCALES_W, "words_s": B.BUF_WORDS_S, "scales_s": B.BUF_SCALES_S}
PER_WORKER = ("x", "m", "u", "delta_w", "words_w", "scales_w")


def _stream():
    return torch.cuda.current_stream().cuda_stream


_GRAD_TYPES = {torch.float32: B.GRAD_F32, torch.float16: B.GRAD_F16, torch.bfloat16: B.GRAD_BF16}


def _grad_ptrs(grads, n, W, dtype=torch.float32):
    if isinstance(grads, torch.Tensor):
        grads = list(grads)
    if len(grads) != W:
        raise ValueError(f"expected {W} gradient tensors, got {len(grads)}")
    for g in grads:
        if not (g.is_cuda and g.dtype == dtype and g.is_contiguous() and g.numel() == n):
            raise ValueError(f"each gradient must be a contiguous {dtype} CUDA tensor of n_params elements")
    return [g.data_ptr() for g in grads]


class Zoa:
    def __init__(self, n_params, W, beta1=0.9, beta2=0.999, eps=1e-8, chunk=4096, allreduce_only=False):
        """allreduce_only: a handle that holds only Algorithm 3's state (zoa_create_allreduce); only
        onebit_allreduce / allreduce_compress / allreduce_average, reads and the checks work on it."""
        self.n, self.W, self.chunk = int(n_params), int(W), int(chunk)
        self.n_chunks = (self.n + self.chunk - 1) // self.chunk
        if allreduce_only:
            self.h = B.zoa_create_allreduce(self.n, self.W, self.chunk)
        else:
            self.h = B.zoa_create(self.n, self.W, beta1, beta2, eps, self.chunk)
        self.grad_dtype = torch.float32

    def close(self):
        if self.h is not None:
            B.zoa_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # -- set-up -------------------------------------------------------------
    def set_params(self, x0):
        x0 = x0.to(device="cuda", dtype=torch.float32).contiguous()
        assert x0.numel() == self.n
        B.zoa_set_params(self.h, x0.data_ptr(), _stream())
        torch.cuda.current_stream().synchronize()   # x0 may be a temporary

    def set_policies(self, var_steps, sync_boundaries, sync_intervals):
        B.zoa_set_var_steps(self.h, list(var_steps))
        B.zoa_set_sync_policy(self.h, list(sync_boundaries), list(sync_intervals))

    def set_pipeline(self, mode):
        """Ring kernels: False = never, True = where shape and problem size allow (default),
        "force" = wherever the shape allows."""
        B.zoa_set_option(self.h, B.OPT_PIPELINE, 2 if mode == "force" else int(bool(mode)))

    def set_grad_dtype(self, dtype):
        """Gradients arrive as torch.float32 (default), torch.float16 or torch.bfloat16."""
        B.zoa_set_option(self.h, B.OPT_GRAD_TYPE, _GRAD_TYPES[dtype])
        self.grad_dtype = dtype

    def sync_due(self, t):
        return B.zoa_sync_due(self.h, t) == 1

    def var_due(self, t):
        return B.zoa_var_due(self.h, t) == 1

    # -- Algorithm 1 --------------------------------------------------------
    def step(self, grads, lr, t):
        B.zoa_step(self.h, _grad_ptrs(grads, self.n, self.W, self.grad_dtype), lr, t, _stream())

    def onebit_reduce(self):
        B.zoa_onebit_reduce(self.h, _stream())

    def onebit_compress(self):
        B.zoa_onebit_compress(self.h, _stream())

    def onebit_average(self):
        B.zoa_onebit_average(self.h, _stream())

    # -- Algorithm 3 on caller-owned buffers ------------------------------------
    def onebit_allreduce(self, z, z_bar):
        """z: W float32 CUDA tensors of n elements (read only), z_bar: float32 CUDA tensor of n elements."""
        B.zoa_onebit_allreduce(self.h, [t.data_ptr() for t in z], z_bar.data_ptr(), _stream())

    def allreduce_compress(self, z):
        B.zoa_allreduce_compress(self.h, [t.data_ptr() for t in z], _stream())

    def allreduce_average(self, z_bar=None):
        B.zoa_allreduce_average(self.h, z_bar.data_ptr() if z_bar is not None else None, _stream())

    def device_view(self, name, worker=0):
        """The state row as a torch tensor that aliases the library's memory (no copy)."""
        which = _NAMES[name]
        ptr, n = B.zoa_get_buffer(self.h, which, worker)
        words = which in B.WORD_BUFFERS

        class _Raw:
            __cuda_array_interface__ = {"shape": (n,), "typestr": "<u4" if words else "<f4",
                                        "data": (ptr, False), "version": 2}
        t = torch.as_tensor(_Raw(), device="cuda")
        return t.view(torch.int32) if words else t

    def step_sync(self, grads, lr, t):
        B.zoa_step_sync(self.h, _grad_ptrs(grads, self.n, self.W, self.grad_dtype), lr, t, _stream())

    def step_auto(self, grads, lr, t):
        B.zoa_step_auto(self.h, _grad_ptrs(grads, self.n, self.W, self.grad_dtype), lr, t, _stream())

    def alg2_step(self, grads, lr, t):
        B.zoa_alg2_step(self.h, _grad_ptrs(grads, self.n, self.W, self.grad_dtype), lr, t, _stream())

    def step_host(self, host_grads, lr, t, host_x_out=None):
        ptrs = [g.data_ptr() for g in host_grads]
        out = host_x_out.data_ptr() if host_x_out is not None else None
        B.zoa_step_host(self.h, ptrs, lr, t, out, _stream())

    # -- state access (synchronous copies) ----------------------------------------
    def read(self, name, worker=0, offset=0, count=None):
        """Copies `count` elements of a state row to a numpy array (default: the live part of the row:
        n parameters, ceil(n / 32) words or n_chunks magnitudes)."""
        which = _NAMES[name]
        if count is None:
            if which in B.WORD_BUFFERS:
                live = (self.n + 31) // 32
            elif name.startswith("scales"):
                live = self.n_chunks
            else:
                live = self.n
            count = live - offset
        out = np.empty(count, np.uint32 if which in B.WORD_BUFFERS else np.float32)
        B.zoa_copy_out(self.h, which, worker, offset, count, out.ctypes.data)
        return out

    def write(self, name, values, worker=0, offset=0):
        which = _NAMES[name]
        values = np.ascontiguousarray(values, np.uint32 if which in B.WORD_BUFFERS else np.float32)
        B.zoa_copy_in(self.h, which, worker, offset, values.size, values.ctypes.data)

    def export_state(self):
        """The whole optimizer state (zoa_export_state) as a numpy byte array."""
        blob = np.empty(B.zoa_state_size(self.h), np.uint8)
        B.zoa_export_state(self.h, blob.ctypes.data, blob.size)
        return blob

    def import_state(self, blob):
        blob = np.ascontiguousarray(blob, np.uint8)
        B.zoa_import_state(self.h, blob.ctypes.data, blob.size)

    def stats(self):
        return B.zoa_get_stats(self.h)

    def check_device(self):
        B.zoa_check_device(self.h)
