"""ctypes binding of ``libcser.so`` - argument marshalling only.

Functions carry the names and argument order of ``include/cser.h``.  Tensors are
passed as raw pointers; torch is used for device memory and streams, nothing
else.  There is no CPU fallback: if the CUDA library has not been built, loading
raises.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcser.so")

STATE_X, STATE_E, STATE_M, STATE_MASK_G, STATE_MASK_R, STATE_T = range(6)

_lib = None


class CSERError(RuntimeError):
    pass


def lib():
    """Load libcser.so once; fail loudly when it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise CSERError(f"{LIB_PATH} not found: build it with "
                        "`python -c 'import __graft_entry__ as g; g.build()'` (needs nvcc)")
    L = ctypes.CDLL(LIB_PATH)
    c = ctypes
    L.cser_create.restype = c.c_void_p
    L.cser_create.argtypes = [c.c_int64, c.c_int32, c.c_int32, c.c_uint32, c.c_uint32, c.c_int32,
                              c.c_float, c.c_float, c.c_uint64]
    L.cser_create_slab.restype = c.c_void_p
    L.cser_create_slab.argtypes = L.cser_create.argtypes + [c.c_int64]
    L.cser_create_ex.restype = c.c_void_p
    L.cser_create_ex.argtypes = L.cser_create_slab.argtypes + [c.c_uint32]
    L.cser_create_wshard.restype = c.c_void_p
    L.cser_create_wshard.argtypes = [c.c_int64, c.c_int32, c.c_int32, c.c_int32, c.c_uint32, c.c_uint32, c.c_int32,
                                     c.c_float, c.c_float, c.c_uint64]
    L.cser_wshard_message_elems.restype = c.c_int64
    L.cser_wshard_message_elems.argtypes = [c.c_void_p, c.c_int]
    L.cser_wshard_pack.restype = c.c_int
    L.cser_wshard_pack.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p]
    L.cser_wshard_apply.restype = c.c_int
    L.cser_wshard_apply.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p]
    L.cser_destroy.restype = None
    L.cser_destroy.argtypes = [c.c_void_p]
    L.cser_set_x0.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p]
    L.cser_step.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p]
    L.cser_step_host.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p]
    L.cser_read_state.argtypes = [c.c_void_p, c.c_int, c.c_void_p, c.c_size_t, c.c_void_p]
    L.cser_write_state.argtypes = [c.c_void_p, c.c_int, c.c_void_p, c.c_size_t, c.c_void_p]
    for name in ("cser_replay_begin", "cser_replay_end"):
        getattr(L, name).restype = c.c_int
        getattr(L, name).argtypes = [c.c_void_p, c.c_void_p]
    L.cser_step_replayable.restype = c.c_int
    L.cser_step_replayable.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p]
    L.cser_read_columns.restype = c.c_int
    L.cser_read_columns.argtypes = [c.c_void_p, c.c_int, c.c_int64, c.c_int64, c.c_void_p, c.c_size_t, c.c_void_p]
    L.cser_set_lr.restype = c.c_int
    L.cser_set_lr.argtypes = [c.c_void_p, c.c_float]
    L.cser_debug_set_masks.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
    L.cser_grbs_mask.argtypes = [c.c_uint64, c.c_uint64, c.c_uint32, c.c_int64, c.c_int64, c.c_uint32,
                                 c.c_void_p, c.c_void_p]
    L.cser_set_timing.argtypes = [c.c_void_p, c.c_int]
    L.cser_last_kernel_ms.argtypes = [c.c_void_p, c.POINTER(c.c_float), c.POINTER(c.c_float)]
    L.cser_launch_count.restype = c.c_int64
    L.cser_launch_count.argtypes = [c.c_void_p]
    L.cser_step_noalloc.restype = c.c_int
    L.cser_step_noalloc.argtypes = [c.c_int64, c.c_int32, c.c_int32, c.c_uint32, c.c_uint32, c.c_int32,
                                    c.c_float, c.c_float, c.c_uint64, c.c_uint64,
                                    c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
    L.cser_debug_stall_next_staged_step.restype = c.c_int
    L.cser_debug_stall_next_staged_step.argtypes = [c.c_void_p, c.c_uint]
    L.cser_last_error.restype = c.c_char_p
    L.cser_last_error.argtypes = []
    L.cser_build_id.restype = c.c_char_p
    L.cser_build_id.argtypes = []
    for name in ("cser_set_x0", "cser_step", "cser_step_host", "cser_read_state", "cser_write_state",
                 "cser_debug_set_masks", "cser_grbs_mask", "cser_set_timing", "cser_last_kernel_ms"):
        getattr(L, name).restype = c.c_int
    _lib = L
    return L


def cser_last_error():
    return lib().cser_last_error().decode()


def cser_build_id():
    return lib().cser_build_id().decode()


def _check(rc, what):
    if rc != 0:
        raise CSERError(f"{what} failed ({rc}): {cser_last_error()}")


def _stream(stream=None):
    """Raw cudaStream_t of `stream`, or of torch's current stream on the current device."""
    if stream is not None:
        return stream.cuda_stream
    return torch._C._cuda_getCurrentRawStream(torch.cuda.current_device())


def _ptr(t):
    return t.data_ptr()


FLAG_NO_ERROR_ARRAY = 1
FLAG_EXACT_COUNT = 2
FLAG_L2_RESIDENT = 4
FLAG_STAGED_SELECTED = 8
FLAG_THREE_KERNELS = 16


def cser_create(d, n_workers, block_size, R1, R2, H, eta, beta, seed, block_begin=0, flags=0):
    h = lib().cser_create_ex(d, n_workers, block_size, R1, R2, H, eta, beta, seed, block_begin, flags)
    if not h:
        raise CSERError(f"cser_create failed: {cser_last_error()}")
    return ctypes.c_void_p(h)


def cser_destroy(h):
    lib().cser_destroy(h)


def cser_set_x0(h, x0, stream=None):
    assert x0.dtype == torch.float32 and x0.is_contiguous()
    _check(lib().cser_set_x0(h, _ptr(x0), _stream(stream)), "cser_set_x0")


def cser_step(h, grad, stream=None):
    assert grad.dtype == torch.float32 and grad.is_contiguous() and grad.is_cuda
    rc = _lib.cser_step(h, grad.data_ptr(), _stream(stream))       # hot path: nothing else per call
    if rc:
        _check(rc, "cser_step")


def cser_step_host(h, grad_host, stream=None):
    assert grad_host.dtype == torch.float32 and grad_host.is_contiguous() and not grad_host.is_cuda
    _check(lib().cser_step_host(h, _ptr(grad_host), _stream(stream)), "cser_step_host")


def cser_read_state(h, which, dst, stream=None):
    _check(lib().cser_read_state(h, which, _ptr(dst), dst.numel() * dst.element_size(), _stream(stream)),
           "cser_read_state")


def cser_replay_begin(h, stream=None):
    _check(lib().cser_replay_begin(h, _stream(stream)), "cser_replay_begin")


def cser_step_replayable(h, grad, stream=None):
    assert grad.dtype == torch.float32 and grad.is_contiguous() and grad.is_cuda
    _check(lib().cser_step_replayable(h, grad.data_ptr(), _stream(stream)), "cser_step_replayable")


def cser_replay_end(h, stream=None):
    _check(lib().cser_replay_end(h, _stream(stream)), "cser_replay_end")


def cser_read_columns(h, which, col_begin, col_count, dst, stream=None):
    assert dst.dtype == torch.float32 and dst.is_contiguous()
    _check(lib().cser_read_columns(h, which, col_begin, col_count, _ptr(dst), dst.numel(), _stream(stream)),
           "cser_read_columns")


def cser_set_lr(h, eta):
    _check(lib().cser_set_lr(h, eta), "cser_set_lr")


def cser_write_state(h, which, src, stream=None):
    assert src.is_contiguous()
    _check(lib().cser_write_state(h, which, _ptr(src), src.numel() * src.element_size(), _stream(stream)),
           "cser_write_state")


def cser_debug_set_masks(h, g_mask, r_mask=None, stream=None):
    _check(lib().cser_debug_set_masks(h, _ptr(g_mask), _ptr(r_mask) if r_mask is not None else None,
                                      _stream(stream)), "cser_debug_set_masks")


def cser_grbs_mask(seed, t, which, block_begin, n_blocks, R, mask_out, stream=None):
    _check(lib().cser_grbs_mask(seed, t, which, block_begin, n_blocks, R, _ptr(mask_out), _stream(stream)),
           "cser_grbs_mask")


def cser_step_noalloc(d, n_workers, block_size, R1, R2, H, eta, beta, seed, t, grad, x, e, m=None, stream=None):
    """One iteration t on arrays the caller owns; the library allocates nothing (see cser.h)."""
    _check(lib().cser_step_noalloc(d, n_workers, block_size, R1, R2, H, eta, beta, seed, t, _ptr(grad),
                                   _ptr(x), _ptr(e), _ptr(m) if m is not None else None, _stream(stream)),
           "cser_step_noalloc")


def cser_set_timing(h, on):
    _check(lib().cser_set_timing(h, int(on)), "cser_set_timing")


def cser_last_kernel_ms(h):
    a, b = ctypes.c_float(), ctypes.c_float()
    _check(lib().cser_last_kernel_ms(h, ctypes.byref(a), ctypes.byref(b)), "cser_last_kernel_ms")
    return a.value, b.value


def cser_launch_count(h):
    return int(lib().cser_launch_count(h))


def cser_create_wshard(d, n_local, n_total, block_size, R1, R2, H, eta, beta, seed):
    h = lib().cser_create_wshard(d, n_local, n_total, block_size, R1, R2, H, eta, beta, seed)
    if not h:
        raise CSERError(f"cser_create_wshard failed: {cser_last_error()}")
    return ctypes.c_void_p(h)


def cser_wshard_message_elems(h, reset_step):
    return int(lib().cser_wshard_message_elems(h, int(bool(reset_step))))


def cser_wshard_pack(h, grad, msg, stream=None):
    assert grad.dtype == torch.float32 and grad.is_contiguous() and grad.is_cuda and msg.dtype == torch.float32
    _check(lib().cser_wshard_pack(h, _ptr(grad), _ptr(msg), msg.numel(), _stream(stream)), "cser_wshard_pack")


def cser_wshard_apply(h, msg, stream=None):
    _check(lib().cser_wshard_apply(h, _ptr(msg), _stream(stream)), "cser_wshard_apply")


class CSER:
    """Convenience owner of one handle (still only marshalling)."""

    def __init__(self, d, n_workers, block_size, R1, R2, H, eta, beta, seed=0, block_begin=0, flags=0):
        self.d, self.n, self.bs, self.beta = int(d), int(n_workers), int(block_size), float(beta)
        self.B = (self.d + self.bs - 1) // self.bs
        self.h = cser_create(d, n_workers, block_size, R1, R2, H, eta, beta, seed, block_begin, flags)

    def close(self):
        if self.h is not None:
            torch.cuda.synchronize()
            cser_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_x0(self, x0):
        cser_set_x0(self.h, x0)

    def step(self, grad):
        cser_step(self.h, grad)

    def step_host(self, grad_host):
        cser_step_host(self.h, grad_host)

    def inject_masks(self, g_mask, r_mask=None):
        cser_debug_set_masks(self.h, g_mask, r_mask)

    def state(self, which, device="cuda"):
        """x / e / m as an [n, d] fp32 tensor, a mask as uint8 [B]."""
        if which in (STATE_X, STATE_E, STATE_M):
            out = torch.empty((self.n, self.d), dtype=torch.float32, device=device)
        else:
            out = torch.empty(self.B, dtype=torch.uint8, device=device)
        cser_read_state(self.h, which, out)
        torch.cuda.current_stream().synchronize()
        return out

    @property
    def t(self):
        out = torch.zeros(1, dtype=torch.int64)
        cser_read_state(self.h, STATE_T, out)
        return int(out.item())


class WorkerShardedCSER(CSER):
    """One rank of the worker-sharded deployment: pack -> all-reduce of the message -> apply.

    torch.distributed is the plumbing for the all-reduce (NCCL between GPUs); with no process
    group, or a group of one, the message is already the global sum.
    """

    def __init__(self, d, n_local, n_total, block_size, R1, R2, H, eta, beta, seed=0, group=None):
        self.d, self.n, self.bs, self.beta = int(d), int(n_local), int(block_size), float(beta)
        self.H, self.group = int(H), group
        self.B = (self.d + self.bs - 1) // self.bs
        self.h = cser_create_wshard(d, n_local, n_total, block_size, R1, R2, H, eta, beta, seed)
        self.msg = torch.empty(max(1, cser_wshard_message_elems(self.h, True)), dtype=torch.float32,
                               device="cuda")
        self._t = 0

    def message_elems(self):
        """Length of the next step's message."""
        return cser_wshard_message_elems(self.h, (self._t + 1) % self.H == 0)

    def pack(self, grad):
        n = self.message_elems()
        cser_wshard_pack(self.h, grad, self.msg)
        self._t += 1
        return self.msg[:n]

    def apply(self):
        cser_wshard_apply(self.h, self.msg)

    def step(self, grad):
        import torch.distributed as dist
        msg = self.pack(grad)
        if dist.is_available() and dist.is_initialized() and dist.get_world_size(self.group) > 1 and msg.numel():
            dist.all_reduce(msg, op=dist.ReduceOp.SUM, group=self.group)
        self.apply()
