"""ctypes binding of libzoa.so: the C ABI of include/zoa.h under the same names.

Argument marshalling only; every step of the method runs in the CUDA kernels.
The shared library must have been built (paper_2202_06009_b200/build.py); there
is no fallback of any kind.
"""
import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libzoa.so")

OK, ERR_ARG, ERR_ALLOC, ERR_CUDA, ERR_STATE, ERR_DEVICE, ERR_NONFINITE = range(7)
(BUF_X, BUF_M, BUF_U, BUF_DELTA_W, BUF_V, BUF_DELTA_S, BUF_X_SYNC,
 BUF_WORDS_W, BUF_SCALES_W, BUF_WORDS_S, BUF_SCALES_S) = range(11)
WORD_BUFFERS = (BUF_WORDS_W, BUF_WORDS_S)


class ZoaError(RuntimeError):
    def __init__(self, status, message):
        super().__init__(f"zoa status {status}: {message}")
        self.status = status


class Stats(C.Structure):
    _fields_ = [("n_steps", C.c_int64), ("n_syncs", C.c_int64), ("n_var_updates", C.c_int64),
                ("n_launches", C.c_int64), ("bits_per_worker", C.c_int64), ("t_last", C.c_int64),
                ("t_sync", C.c_int64), ("gamma_sum", C.c_double)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2202_06009_b200.build` "
                          "(or __graft_entry__.build()); this package has no CPU path")
    lib = C.CDLL(LIB_PATH)
    H, p = C.c_void_p, C.c_void_p
    sigs = {
        "zoa_create": ([C.POINTER(H), C.c_size_t, C.c_int, C.c_float, C.c_float, C.c_float, C.c_int], C.c_int),
        "zoa_destroy": ([H], C.c_int),
        "zoa_set_params": ([H, p, p], C.c_int),
        "zoa_set_var_steps": ([H, C.POINTER(C.c_int64), C.c_size_t], C.c_int),
        "zoa_set_var_policy": ([H, C.POINTER(C.c_int64), C.c_size_t], C.c_int),
        "zoa_set_var_policy_doubling": ([H, C.c_int, C.c_int64], C.c_int),
        "zoa_set_sync_policy": ([H, C.POINTER(C.c_int64), C.POINTER(C.c_int32), C.c_size_t], C.c_int),
        "zoa_policy_var_steps": ([C.c_int, C.c_int64, C.POINTER(C.c_int64), C.c_size_t], C.c_size_t),
        "zoa_policy_sync_pieces": ([C.c_int64, C.c_int64, C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_int32),
                                    C.c_size_t], C.c_size_t),
        "zoa_set_sync_policy_doubling": ([H, C.c_int64, C.c_int64, C.c_int32, C.c_int], C.c_int),
        "zoa_sync_due": ([H, C.c_int64], C.c_int),
        "zoa_var_due": ([H, C.c_int64], C.c_int),
        "zoa_step": ([H, C.POINTER(p), C.c_float, C.c_int64, p], C.c_int),
        "zoa_onebit_reduce": ([H, p], C.c_int),
        "zoa_onebit_compress": ([H, p], C.c_int),
        "zoa_onebit_average": ([H, p], C.c_int),
        "zoa_create_allreduce": ([C.POINTER(H), C.c_size_t, C.c_int, C.c_int], C.c_int),
        "zoa_onebit_allreduce": ([H, C.POINTER(p), p, p], C.c_int),
        "zoa_allreduce_compress": ([H, C.POINTER(p), p], C.c_int),
        "zoa_allreduce_average": ([H, p, p], C.c_int),
        "zoa_dist_server_range": ([H, p, C.c_size_t, p, C.c_size_t, C.c_int, C.c_int64, C.c_int64, p], C.c_int),
        "zoa_dist_apply": ([H, p], C.c_int),
        "zoa_dist_variance": ([H, p, p], C.c_int),
        "zoa_dist_pack_push": ([H, C.c_int, C.POINTER(C.c_int64), C.POINTER(p), C.POINTER(p), p], C.c_int),
        "zoa_dist_step_pack_push": ([H, p, C.c_float, C.c_int64, C.c_int, C.POINTER(C.c_int64), C.POINTER(p), C.POINTER(p), p], C.c_int),
        "zoa_dist_server_push": ([H, p, C.c_size_t, p, C.c_size_t, C.c_int, C.c_int64, C.c_int64, C.c_int, C.POINTER(p), C.POINTER(p), p], C.c_int),
        "zoa_step_sync": ([H, C.POINTER(p), C.c_float, C.c_int64, p], C.c_int),
        "zoa_step_auto": ([H, C.POINTER(p), C.c_float, C.c_int64, p], C.c_int),
        "zoa_alg2_step": ([H, C.POINTER(p), C.c_float, C.c_int64, p], C.c_int),
        "zoa_step_host": ([H, C.POINTER(p), C.c_float, C.c_int64, p, p], C.c_int),
        "zoa_get_buffer": ([H, C.c_int, C.c_int, C.POINTER(p), C.POINTER(C.c_size_t)], C.c_int),
        "zoa_get_ptr": ([H, C.c_int, C.c_int, C.POINTER(p), C.POINTER(C.c_size_t)], C.c_int),
        "zoa_state_size": ([H, C.POINTER(C.c_size_t)], C.c_int),
        "zoa_export_state": ([H, p, C.c_size_t], C.c_int),
        "zoa_import_state": ([H, p, C.c_size_t], C.c_int),
        "zoa_copy_out": ([H, C.c_int, C.c_int, C.c_size_t, C.c_size_t, p], C.c_int),
        "zoa_copy_in": ([H, C.c_int, C.c_int, C.c_size_t, C.c_size_t, p], C.c_int),
        "zoa_set_scalars": ([H, C.c_double, C.c_int64, C.c_int64], C.c_int),
        "zoa_get_stats": ([H, C.POINTER(Stats)], C.c_int),
        "zoa_check_device": ([H], C.c_int),
        "zoa_check_finite": ([H, C.POINTER(C.c_int64)], C.c_int),
        "zoa_last_error": ([H], C.c_char_p),
        "zoa_set_option": ([H, C.c_int, C.c_int], C.c_int),
        "zoa_onebit_allreduce_static": ([C.POINTER(p), C.POINTER(p), p, p, C.c_size_t, C.c_int, C.c_int, p], C.c_int),
        "zoa_static_scratch_slots": ([], C.c_size_t),
        "zoa_static_last_error": ([], C.c_char_p),
    }
    for name, (argtypes, restype) in sigs.items():
        fn = getattr(lib, name)
        fn.argtypes, fn.restype = argtypes, restype
    return lib, tuple(sigs)


lib, EXPORTS = _load()


def _check(handle, status):
    if status != OK:
        raise ZoaError(status, lib.zoa_last_error(handle).decode())


def _ptr_array(ptrs):
    return (C.c_void_p * len(ptrs))(*ptrs)


# -- the C calls under their own names (handle = ctypes.c_void_p) ---------------
def zoa_create(n_params, W, beta1, beta2, eps, chunk):
    h = C.c_void_p()
    _check(None, lib.zoa_create(C.byref(h), n_params, W, beta1, beta2, eps, chunk))
    return h


def zoa_destroy(h):
    _check(None, lib.zoa_destroy(h))


def zoa_set_params(h, x0_ptr, stream=0):
    _check(h, lib.zoa_set_params(h, x0_ptr, stream))


def zoa_set_var_steps(h, steps):
    arr = (C.c_int64 * len(steps))(*steps)
    _check(h, lib.zoa_set_var_steps(h, arr, len(steps)))


def zoa_set_var_policy_doubling(h, kappa, freeze_at):
    _check(h, lib.zoa_set_var_policy_doubling(h, kappa, freeze_at))


def zoa_set_sync_policy(h, boundaries, intervals):
    b = (C.c_int64 * len(boundaries))(*boundaries)
    k = (C.c_int32 * len(intervals))(*intervals)
    _check(h, lib.zoa_set_sync_policy(h, b, k, len(boundaries)))


def zoa_policy_var_steps(kappa, freeze_at):
    n = lib.zoa_policy_var_steps(kappa, freeze_at, None, 0)
    out = (C.c_int64 * n)()
    lib.zoa_policy_var_steps(kappa, freeze_at, out, n)
    return list(out)


def zoa_policy_sync_pieces(warmup, double_every, max_interval):
    n = lib.zoa_policy_sync_pieces(warmup, double_every, max_interval, None, None, 0)
    b, k = (C.c_int64 * n)(), (C.c_int32 * n)()
    lib.zoa_policy_sync_pieces(warmup, double_every, max_interval, b, k, n)
    return list(b), list(k)


def zoa_set_sync_policy_doubling(h, warmup, double_every, max_interval, freeze_variance=True):
    _check(h, lib.zoa_set_sync_policy_doubling(h, warmup, double_every, max_interval, int(bool(freeze_variance))))


def zoa_sync_due(h, t):
    return lib.zoa_sync_due(h, t)


def zoa_var_due(h, t):
    return lib.zoa_var_due(h, t)


def zoa_step(h, grad_ptrs, lr, t, stream=0):
    _check(h, lib.zoa_step(h, _ptr_array(grad_ptrs), lr, t, stream))


def zoa_onebit_reduce(h, stream=0):
    _check(h, lib.zoa_onebit_reduce(h, stream))


def zoa_onebit_compress(h, stream=0):
    _check(h, lib.zoa_onebit_compress(h, stream))


def zoa_onebit_average(h, stream=0):
    _check(h, lib.zoa_onebit_average(h, stream))


def zoa_create_allreduce(n_params, W, chunk):
    h = C.c_void_p()
    _check(None, lib.zoa_create_allreduce(C.byref(h), n_params, W, chunk))
    return h


def zoa_onebit_allreduce(h, z_ptrs, z_bar_ptr, stream=0):
    _check(h, lib.zoa_onebit_allreduce(h, _ptr_array(z_ptrs), z_bar_ptr, stream))


def zoa_allreduce_compress(h, z_ptrs, stream=0):
    _check(h, lib.zoa_allreduce_compress(h, _ptr_array(z_ptrs), stream))


def zoa_allreduce_average(h, z_bar_ptr, stream=0):
    _check(h, lib.zoa_allreduce_average(h, z_bar_ptr, stream))


def zoa_dist_server_range(h, words_ptr, words_stride, scales_ptr, scales_stride, W_total, first_chunk, n_chunks, stream=0):
    _check(h, lib.zoa_dist_server_range(h, words_ptr, words_stride, scales_ptr, scales_stride, W_total,
                                        first_chunk, n_chunks, stream))


def zoa_dist_apply(h, stream=0):
    _check(h, lib.zoa_dist_apply(h, stream))


def zoa_dist_variance(h, g_bar_ptr, stream=0):
    _check(h, lib.zoa_dist_variance(h, g_bar_ptr, stream))


def _i64_array(values):
    return (C.c_int64 * len(values))(*values)


def zoa_dist_pack_push(h, chunk_begin, peer_words, peer_scales, stream=0):
    world = len(peer_words)
    _check(h, lib.zoa_dist_pack_push(h, world, _i64_array(chunk_begin), _ptr_array(peer_words), _ptr_array(peer_scales), stream))


def zoa_dist_step_pack_push(h, grad_ptr, lr, t, chunk_begin, peer_words, peer_scales, stream=0):
    world = len(peer_words)
    _check(h, lib.zoa_dist_step_pack_push(h, grad_ptr, lr, t, world, _i64_array(chunk_begin), _ptr_array(peer_words),
                                          _ptr_array(peer_scales), stream))


def zoa_dist_server_push(h, words_ptr, words_stride, scales_ptr, scales_stride, W_total, first_chunk, n_chunks,
                         peer_words_s, peer_scales_s, stream=0):
    _check(h, lib.zoa_dist_server_push(h, words_ptr, words_stride, scales_ptr, scales_stride, W_total, first_chunk,
                                       n_chunks, len(peer_words_s), _ptr_array(peer_words_s), _ptr_array(peer_scales_s), stream))


def zoa_step_sync(h, grad_ptrs, lr, t, stream=0):
    _check(h, lib.zoa_step_sync(h, _ptr_array(grad_ptrs), lr, t, stream))


def zoa_step_auto(h, grad_ptrs, lr, t, stream=0):
    _check(h, lib.zoa_step_auto(h, _ptr_array(grad_ptrs), lr, t, stream))


def zoa_alg2_step(h, grad_ptrs, lr, t, stream=0):
    _check(h, lib.zoa_alg2_step(h, _ptr_array(grad_ptrs), lr, t, stream))


def zoa_step_host(h, host_grad_ptrs, lr, t, host_x_out_ptr=None, stream=0):
    _check(h, lib.zoa_step_host(h, _ptr_array(host_grad_ptrs), lr, t, host_x_out_ptr, stream))


def zoa_get_buffer(h, which, worker=0):
    ptr, n = C.c_void_p(), C.c_size_t()
    _check(h, lib.zoa_get_buffer(h, which, worker, C.byref(ptr), C.byref(n)))
    return ptr.value, n.value


def zoa_get_ptr(h, what, worker=0):
    ptr, n = C.c_void_p(), C.c_size_t()
    _check(h, lib.zoa_get_ptr(h, what, worker, C.byref(ptr), C.byref(n)))
    return ptr.value, n.value


def zoa_set_var_policy(h, steps):
    arr = (C.c_int64 * len(steps))(*steps)
    _check(h, lib.zoa_set_var_policy(h, arr, len(steps)))


def zoa_state_size(h):
    n = C.c_size_t()
    _check(h, lib.zoa_state_size(h, C.byref(n)))
    return n.value


def zoa_export_state(h, host_ptr, nbytes):
    _check(h, lib.zoa_export_state(h, host_ptr, nbytes))


def zoa_import_state(h, host_ptr, nbytes):
    _check(h, lib.zoa_import_state(h, host_ptr, nbytes))


def zoa_copy_out(h, which, worker, offset, count, host_ptr):
    _check(h, lib.zoa_copy_out(h, which, worker, offset, count, host_ptr))


def zoa_copy_in(h, which, worker, offset, count, host_ptr):
    _check(h, lib.zoa_copy_in(h, which, worker, offset, count, host_ptr))


def zoa_set_scalars(h, gamma_sum, t_sync, t_last):
    _check(h, lib.zoa_set_scalars(h, gamma_sum, t_sync, t_last))


def zoa_get_stats(h):
    s = Stats()
    _check(h, lib.zoa_get_stats(h, C.byref(s)))
    return {name: getattr(s, name) for name, _ in Stats._fields_}


OPT_PIPELINE, OPT_WAIT_LIMIT_MS, OPT_TEST_STOP_AFTER_TILES, OPT_GRAD_TYPE = 1, 2, 3, 4
GRAD_F32, GRAD_F16, GRAD_BF16 = 0, 1, 2


def zoa_set_option(h, option, value):
    _check(h, lib.zoa_set_option(h, option, value))


def zoa_check_finite(h):
    """Number of NaN / infinite values in the float state (0 = clean); never raises for a non-zero count."""
    n = C.c_int64()
    status = lib.zoa_check_finite(h, C.byref(n))
    if status not in (OK, ERR_NONFINITE):
        _check(h, status)
    return n.value


def zoa_check_device(h):
    _check(h, lib.zoa_check_device(h))


def zoa_onebit_allreduce_static(z_ptrs, delta_w_ptrs, delta_s_ptr, z_bar_ptr, n, W, chunk, stream=0):
    """Algorithm 3 on caller-owned device buffers, allocating nothing (see include/zoa.h)."""
    status = lib.zoa_onebit_allreduce_static(_ptr_array(z_ptrs), _ptr_array(delta_w_ptrs), delta_s_ptr,
                                             z_bar_ptr, n, W, chunk, stream)
    if status != OK:
        raise ZoaError(status, lib.zoa_static_last_error().decode())


def zoa_static_scratch_slots():
    return lib.zoa_static_scratch_slots()
