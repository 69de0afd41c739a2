"""Thin Python binding over the C ABI of libtemplora.so (include/templora.h).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  torch provides device memory and streams.  The functions carry the
names of the C entry points.  There is no CPU fallback: importing this module
without the compiled library raises.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtemplora.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)
F32, BF16 = 0, 1

EXPORTS = [
    "templora_workspace_bytes", "templora_update_block_workspace_bytes", "templora_linear_fwd",
    "templora_linear_bwd", "templora_adamw_step", "templora_decode_fwd", "templora_update_block",
    "templora_status_string", "templora_read_device_status", "templora_set_kernel_path",
    "templora_timing_enable", "templora_timing_read", "templora_decode_fwd_noalloc",
    "templora_decode_block_workspace_bytes", "templora_decode_block_fwd", "templora_update_block_batched",
    "templora_set_stream_sm_limit", "templora_selftest_bounded_wait", "templora_lr_at_step",
    "templora_update_block_warmup", "templora_swiglu_fwd", "templora_swiglu_bwd", "templora_rmsnorm_fwd",
    "templora_rmsnorm_bwd", "templora_decode_fwd_noalloc_status", "templora_update_mlp",
    "templora_update_mlp_workspace_bytes", "templora_sm_partition_create", "templora_sm_partition_destroy",
    "templora_update_attn_in",
]
NOALLOC_SCRATCH_BYTES = 8 << 20
(KIND_TC_MAIN, KIND_TC_SKINNY, KIND_TC_DECODE, KIND_REDUCE, KIND_ADAMW, KIND_SIMT, KIND_DECODE_FINISH, KIND_DROPOUT,
 KIND_TC_DROPOUT_TERM, KIND_BLOCK_OPS) = range(10)
N_KINDS = 10


class SmPartition(C.Structure):
    """templora_sm_partition_t: two streams whose kernels run on disjoint groups of SMs."""
    _fields_ = [("handle", C.c_void_p), ("stream_first", C.c_void_p), ("stream_rest", C.c_void_p),
                ("sms_first", C.c_int32), ("sms_rest", C.c_int32)]


class LinearDesc(C.Structure):
    _fields_ = [("d_in", C.c_int32), ("d_out", C.c_int32), ("r", C.c_int32), ("s", C.c_float),
                ("dtype", C.c_int32), ("W0", C.c_void_p), ("A", C.c_void_p), ("B", C.c_void_p),
                ("dropout_p", C.c_float), ("input_group", C.c_int32), ("dropout_seed", C.c_uint64),
                ("dropout_offset", C.c_uint64)]


class ParamDesc(C.Structure):
    _fields_ = [("n", C.c_int64), ("master", C.c_void_p), ("m", C.c_void_p), ("v", C.c_void_p),
                ("work", C.c_void_p), ("grad", C.c_void_p)]


class TemploraError(RuntimeError):
    def __init__(self, code, what):
        self.code = code
        super().__init__(f"{what}: {status_string(code)} (status {code})")


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2401_11504_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, f32, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t
    LP, PP = C.POINTER(LinearDesc), C.POINTER(ParamDesc)
    lib.templora_workspace_bytes.restype = sz
    lib.templora_workspace_bytes.argtypes = [LP, i32]
    lib.templora_update_block_workspace_bytes.restype = sz
    lib.templora_update_block_workspace_bytes.argtypes = [LP, i32, i32]
    lib.templora_linear_fwd.restype = i32
    lib.templora_linear_fwd.argtypes = [LP, i32, vp, vp, vp, vp, sz, vp]
    lib.templora_linear_bwd.restype = i32
    lib.templora_linear_bwd.argtypes = [LP, i32, vp, vp, vp, vp, vp, vp, i32, vp, sz, vp]
    lib.templora_adamw_step.restype = i32
    lib.templora_adamw_step.argtypes = [PP, i32, f32, f32, f32, f32, f32, i64, i32, vp]
    lib.templora_decode_fwd.restype = i32
    lib.templora_decode_fwd.argtypes = [LP, i32, vp, vp, vp, sz, vp]
    lib.templora_update_block.restype = i32
    lib.templora_update_block.argtypes = [LP, PP, PP, i32, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp),
                                          C.POINTER(vp), i32, f32, f32, f32, f32, f32, C.POINTER(i64), vp, sz, vp]
    lib.templora_update_block_batched.restype = i32
    lib.templora_update_block_batched.argtypes = [LP, PP, PP, i32, i32, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp),
                                                  C.POINTER(vp), i32, f32, f32, f32, f32, f32, C.POINTER(i64), vp, sz, vp]
    lib.templora_update_block_warmup.restype = i32
    lib.templora_update_block_warmup.argtypes = [LP, PP, PP, i32, i32, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp),
                                                 C.POINTER(vp), i32, f32, i64, f32, f32, f32, f32, C.POINTER(i64), vp, sz, vp]
    lib.templora_update_mlp_workspace_bytes.restype = sz
    lib.templora_update_mlp_workspace_bytes.argtypes = [LP, i32]
    lib.templora_update_mlp.restype = i32
    lib.templora_update_mlp.argtypes = [LP, PP, PP, i32, vp, vp, vp, vp, vp, vp, vp, i32, f32, f32, f32, f32, f32,
                                        C.POINTER(i64), vp, sz, vp]
    lib.templora_update_attn_in.restype = i32
    lib.templora_update_attn_in.argtypes = [LP, PP, PP, i32, i32, vp, vp, f32, C.POINTER(vp), vp, C.POINTER(vp), vp, vp,
                                            i32, f32, f32, f32, f32, f32, C.POINTER(i64), vp, sz, vp]
    lib.templora_swiglu_fwd.restype = i32
    lib.templora_swiglu_fwd.argtypes = [i64, i32, vp, vp, vp, vp]
    lib.templora_swiglu_bwd.restype = i32
    lib.templora_swiglu_bwd.argtypes = [i64, i32, vp, vp, vp, vp, vp, vp]
    lib.templora_rmsnorm_fwd.restype = i32
    lib.templora_rmsnorm_fwd.argtypes = [i32, i32, i32, vp, vp, f32, vp, vp]
    lib.templora_rmsnorm_bwd.restype = i32
    lib.templora_rmsnorm_bwd.argtypes = [i32, i32, i32, vp, vp, vp, f32, vp, vp]
    lib.templora_lr_at_step.restype = f32
    lib.templora_lr_at_step.argtypes = [f32, i64, i64]
    lib.templora_selftest_bounded_wait.restype = i32
    lib.templora_selftest_bounded_wait.argtypes = [vp, sz, i32, vp]
    lib.templora_set_stream_sm_limit.restype = i32
    lib.templora_set_stream_sm_limit.argtypes = [vp, i32]
    lib.templora_sm_partition_create.restype = i32
    lib.templora_sm_partition_create.argtypes = [i32, C.POINTER(SmPartition)]
    lib.templora_sm_partition_destroy.restype = i32
    lib.templora_sm_partition_destroy.argtypes = [C.POINTER(SmPartition)]
    lib.templora_status_string.restype = C.c_char_p
    lib.templora_status_string.argtypes = [i32]
    lib.templora_read_device_status.restype = i32
    lib.templora_read_device_status.argtypes = [vp, vp, C.POINTER(i32), C.POINTER(i32)]
    lib.templora_set_kernel_path.restype = i32
    lib.templora_set_kernel_path.argtypes = [i32]
    lib.templora_decode_block_workspace_bytes.restype = sz
    lib.templora_decode_block_workspace_bytes.argtypes = [LP, i32]
    lib.templora_decode_block_fwd.restype = i32
    lib.templora_decode_block_fwd.argtypes = [LP, i32, i32, C.POINTER(vp), C.POINTER(vp), vp, sz, vp]
    lib.templora_decode_fwd_noalloc.restype = i32
    lib.templora_decode_fwd_noalloc.argtypes = [LP, i32, vp, vp, vp]
    lib.templora_decode_fwd_noalloc_status.restype = i32
    lib.templora_decode_fwd_noalloc_status.argtypes = [vp, C.POINTER(i32), C.POINTER(i32)]
    lib.templora_timing_enable.restype = None
    lib.templora_timing_enable.argtypes = [i32]
    lib.templora_timing_read.restype = i32
    lib.templora_timing_read.argtypes = [i32, C.POINTER(C.c_double), C.POINTER(i64), C.POINTER(i64), i32]
    return lib


lib = _load()


def status_string(code):
    return lib.templora_status_string(int(code)).decode()


def _check(code, what):
    if code != OK:
        raise TemploraError(code, what)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def dtype_code(t):
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported storage dtype {t.dtype}")


def linear_desc(W0, A, B, s, dropout_p=0.0, dropout_seed=0, dropout_offset=0, input_group=0):
    """templora_linear_t for contiguous device tensors W0 [d_out,d_in], A [r,d_in], B [d_out,r]."""
    for t in (W0, A, B):
        if not t.is_contiguous():
            raise ValueError("W0, A and B must be contiguous")
    d_out, d_in = W0.shape
    r = A.shape[0]
    if tuple(A.shape) != (r, d_in) or tuple(B.shape) != (d_out, r) or A.dtype != W0.dtype or B.dtype != W0.dtype:
        raise ValueError("shape/dtype mismatch between W0, A and B")
    desc = LinearDesc(d_in, d_out, r, float(s), dtype_code(W0), W0.data_ptr(), A.data_ptr(), B.data_ptr(),
                      float(dropout_p), int(input_group), int(dropout_seed), int(dropout_offset))
    desc._keep = (W0, A, B)  # the descriptor holds raw pointers: keep the tensors alive with it
    return desc


def param_desc(master, m, v, grad, work=None):
    desc = ParamDesc(master.numel(), master.data_ptr(), m.data_ptr(), v.data_ptr(),
                     0 if work is None else work.data_ptr(), grad.data_ptr())
    desc._keep = (master, m, v, grad, work)
    return desc


def templora_workspace_bytes(lin, T):
    return int(lib.templora_workspace_bytes(C.byref(lin), int(T)))


def templora_update_block_workspace_bytes(lins, T):
    arr = (LinearDesc * len(lins))(*lins)
    return int(lib.templora_update_block_workspace_bytes(arr, len(lins), int(T)))


def alloc_workspace(nbytes, device="cuda"):
    """Zeroed workspace (the head holds the device status record)."""
    if nbytes <= 0:
        raise ValueError("workspace size query failed (invalid projection?)")
    return torch.zeros(int(nbytes), dtype=torch.uint8, device=device)


def templora_linear_fwd(lin, x, y, ws, U_save=None, stream=None):
    _check(lib.templora_linear_fwd(C.byref(lin), x.shape[0], _ptr(x), _ptr(y), _ptr(U_save), _ptr(ws),
                                   ws.numel(), _stream(stream)), "templora_linear_fwd")


def templora_linear_bwd(lin, x, dY, dX, dA, dB, ws, U_saved=None, accumulate=False, stream=None):
    _check(lib.templora_linear_bwd(C.byref(lin), x.shape[0], _ptr(x), _ptr(dY), _ptr(U_saved), _ptr(dX), _ptr(dA),
                                   _ptr(dB), int(bool(accumulate)), _ptr(ws), ws.numel(), _stream(stream)),
           "templora_linear_bwd")


def templora_adamw_step(params, lr, beta1, beta2, eps, weight_decay, step, work_dtype=BF16, stream=None):
    arr = (ParamDesc * len(params))(*params)
    _check(lib.templora_adamw_step(arr, len(params), lr, beta1, beta2, eps, weight_decay, int(step),
                                   int(work_dtype), _stream(stream)), "templora_adamw_step")


def templora_decode_fwd(lin, x, y, ws, stream=None):
    _check(lib.templora_decode_fwd(C.byref(lin), x.shape[0], _ptr(x), _ptr(y), _ptr(ws), ws.numel(),
                                   _stream(stream)), "templora_decode_fwd")


class UpdateBlockArgs:
    """Marshalled argument arrays of templora_update_block, built once and reusable."""

    def __init__(self, lins, A_states, B_states, xs, dYs, ys, dXs=None):
        n = len(lins)
        self.n = n
        self.T = xs[0].shape[0]
        self.lins = (LinearDesc * n)(*lins)
        self.A = (ParamDesc * n)(*A_states)
        self.B = (ParamDesc * n)(*B_states)
        vp = C.c_void_p
        self.x = (vp * n)(*[t.data_ptr() for t in xs])
        self.dY = (vp * n)(*[t.data_ptr() for t in dYs])
        self.y = (vp * n)(*[t.data_ptr() for t in ys])
        self.dX = None if dXs is None else (vp * n)(*[0 if t is None else t.data_ptr() for t in dXs])
        self._keep = (lins, A_states, B_states, xs, dYs, ys, dXs)


def templora_update_block(args, epochs, lr, beta1, beta2, eps, weight_decay, step, ws, stream=None):
    """Runs the chunk update; returns the new optimizer step count."""
    st = C.c_int64(int(step))
    _check(lib.templora_update_block(args.lins, args.A, args.B, args.n, args.T, args.x, args.dY, args.y, args.dX,
                                     int(epochs), lr, beta1, beta2, eps, weight_decay, C.byref(st), _ptr(ws),
                                     ws.numel(), _stream(stream)), "templora_update_block")
    return st.value


def templora_update_block_batched(args, batch_tokens, epochs, lr, beta1, beta2, eps, weight_decay, step, ws,
                                  stream=None):
    """Chunk update with one optimizer step per batch of batch_tokens rows; returns the new step count."""
    st = C.c_int64(int(step))
    _check(lib.templora_update_block_batched(args.lins, args.A, args.B, args.n, args.T, int(batch_tokens), args.x,
                                             args.dY, args.y, args.dX, int(epochs), lr, beta1, beta2, eps,
                                             weight_decay, C.byref(st), _ptr(ws), ws.numel(), _stream(stream)),
           "templora_update_block_batched")
    return st.value


def templora_update_block_warmup(args, batch_tokens, epochs, lr, warmup_steps, beta1, beta2, eps, weight_decay, step, ws,
                                 stream=None):
    """Batched chunk update with the linear learning-rate warm-up applied per optimizer step."""
    st = C.c_int64(int(step))
    _check(lib.templora_update_block_warmup(args.lins, args.A, args.B, args.n, args.T, int(batch_tokens), args.x,
                                            args.dY, args.y, args.dX, int(epochs), lr, int(warmup_steps), beta1, beta2,
                                            eps, weight_decay, C.byref(st), _ptr(ws), ws.numel(), _stream(stream)),
           "templora_update_block_warmup")
    return st.value


def templora_update_mlp_workspace_bytes(lins, T):
    arr = (LinearDesc * 3)(*lins)
    return int(lib.templora_update_mlp_workspace_bytes(arr, int(T)))


def templora_update_mlp(lins, A_states, B_states, x, dY, gate, up, h, y, dX, epochs, lr, beta1, beta2, eps, weight_decay,
                        step, ws, stream=None):
    """Chunk update of a block's MLP (lins, A_states, B_states: gate, up, down); returns the new step count."""
    st = C.c_int64(int(step))
    _check(lib.templora_update_mlp((LinearDesc * 3)(*lins), (ParamDesc * 3)(*A_states), (ParamDesc * 3)(*B_states),
                                   x.shape[0], _ptr(x), _ptr(dY), _ptr(gate), _ptr(up), _ptr(h), _ptr(y), _ptr(dX),
                                   int(epochs), lr, beta1, beta2, eps, weight_decay, C.byref(st), _ptr(ws), ws.numel(),
                                   _stream(stream)), "templora_update_mlp")
    return st.value


def templora_update_attn_in(lins, A_states, B_states, x, norm_weight, norm_eps, dYs, xn, ys, dXn, dX, epochs, lr, beta1,
                            beta2, eps, weight_decay, step, ws, stream=None):
    """Chunk update of the projections behind a block's input norm (q, k, v): RMSNorm, the projections on the shared
    normalised input with one summed input gradient, the norm's backward; returns the new step count."""
    n = len(lins)
    st = C.c_int64(int(step))
    vp = C.c_void_p
    dy_arr = (vp * n)(*[t.data_ptr() for t in dYs])
    y_arr = (vp * n)(*[t.data_ptr() for t in ys])
    _check(lib.templora_update_attn_in((LinearDesc * n)(*lins), (ParamDesc * n)(*A_states), (ParamDesc * n)(*B_states), n,
                                       x.shape[0], _ptr(x), _ptr(norm_weight), norm_eps, dy_arr, _ptr(xn), y_arr, _ptr(dXn),
                                       _ptr(dX), int(epochs), lr, beta1, beta2, eps, weight_decay, C.byref(st), _ptr(ws),
                                       ws.numel(), _stream(stream)), "templora_update_attn_in")
    return st.value


def templora_swiglu_fwd(gate, up, h, stream=None):
    """h = SiLU(gate) * up, element-wise over contiguous tensors of one shape and dtype."""
    _check(lib.templora_swiglu_fwd(gate.numel(), dtype_code(gate), _ptr(gate), _ptr(up), _ptr(h), _stream(stream)),
           "templora_swiglu_fwd")


def templora_swiglu_bwd(gate, up, dh, dgate, dup, stream=None):
    _check(lib.templora_swiglu_bwd(gate.numel(), dtype_code(gate), _ptr(gate), _ptr(up), _ptr(dh), _ptr(dgate), _ptr(dup),
                                   _stream(stream)), "templora_swiglu_bwd")


def templora_rmsnorm_fwd(x, w, eps, y, stream=None):
    """y = x / sqrt(mean(x^2) + eps) * w over the rows of a contiguous [T, d] tensor."""
    _check(lib.templora_rmsnorm_fwd(x.shape[0], x.shape[1], dtype_code(x), _ptr(x), _ptr(w), eps, _ptr(y),
                                    _stream(stream)), "templora_rmsnorm_fwd")


def templora_rmsnorm_bwd(x, w, dy, eps, dx, stream=None):
    _check(lib.templora_rmsnorm_bwd(x.shape[0], x.shape[1], dtype_code(x), _ptr(x), _ptr(w), _ptr(dy), eps, _ptr(dx),
                                    _stream(stream)), "templora_rmsnorm_bwd")


def templora_lr_at_step(lr, step, warmup_steps):
    return float(lib.templora_lr_at_step(lr, int(step), int(warmup_steps)))


def templora_read_device_status(ws, stream=None):
    code, where = C.c_int32(0), C.c_int32(0)
    _check(lib.templora_read_device_status(_ptr(ws), _stream(stream), C.byref(code), C.byref(where)),
           "templora_read_device_status")
    return code.value, where.value


def templora_set_kernel_path(mode):
    return int(lib.templora_set_kernel_path(int(mode)))


def templora_timing_enable(kinds):
    """kinds: iterable of kernel classes to time, True for all, False/None for none."""
    if kinds is True:
        mask = -1
    elif not kinds:
        mask = 0
    else:
        mask = 0
        for k in kinds:
            mask |= 1 << int(k)
    lib.templora_timing_enable(mask)


def templora_timing_read(kind, reset=False):
    """-> (total_ms, timed_launches, all_launches) of one kernel class."""
    ms, timed, allc = C.c_double(0.0), C.c_int64(0), C.c_int64(0)
    _check(lib.templora_timing_read(int(kind), C.byref(ms), C.byref(timed), C.byref(allc), int(bool(reset))),
           "templora_timing_read")
    return ms.value, timed.value, allc.value


def templora_decode_fwd_noalloc(lin, x, y, stream=None):
    """Decode-time forward without a caller workspace: for hosts that may not allocate device
    memory.  Scratch is a fixed array inside the library (NOALLOC_SCRATCH_BYTES per GPU), shared by
    all calls on the device, so calls that could overlap on the GPU must be serialised."""
    _check(lib.templora_decode_fwd_noalloc(C.byref(lin), x.shape[0], _ptr(x), _ptr(y), _stream(stream)),
           "templora_decode_fwd_noalloc")


def templora_decode_fwd_noalloc_status(stream=None):
    """(code, where) of the most recent templora_decode_fwd_noalloc call on this device; synchronises the stream."""
    code, where = C.c_int32(0), C.c_int32(0)
    _check(lib.templora_decode_fwd_noalloc_status(_stream(stream), C.byref(code), C.byref(where)),
           "templora_decode_fwd_noalloc_status")
    return code.value, where.value


def templora_decode_block_workspace_bytes(lins):
    arr = (LinearDesc * len(lins))(*lins)
    return int(lib.templora_decode_block_workspace_bytes(arr, len(lins)))


class DecodeBlockArgs:
    """Marshalled argument arrays of templora_decode_block_fwd, built once and reusable."""

    def __init__(self, lins, xs, ys):
        n = len(lins)
        self.n, self.n_tokens = n, xs[0].shape[0]
        self.lins = (LinearDesc * n)(*lins)
        self.x = (C.c_void_p * n)(*[t.data_ptr() for t in xs])
        self.y = (C.c_void_p * n)(*[t.data_ptr() for t in ys])
        self._keep = (lins, xs, ys)


def templora_decode_block_fwd(args, ws, stream=None):
    _check(lib.templora_decode_block_fwd(args.lins, args.n, args.n_tokens, args.x, args.y, _ptr(ws), ws.numel(),
                                         _stream(stream)), "templora_decode_block_fwd")


def templora_set_stream_sm_limit(stream, max_sms):
    """Cap the SMs the persistent kernels use on `stream` (0 = no cap)."""
    _check(lib.templora_set_stream_sm_limit(_stream(stream), int(max_sms)), "templora_set_stream_sm_limit")


def templora_sm_partition_create(first_sms):
    """Split the current device's SMs into two groups with one stream each; returns the filled SmPartition
    (wrap its streams with torch.cuda.ExternalStream to use them from torch)."""
    part = SmPartition()
    _check(lib.templora_sm_partition_create(int(first_sms), C.byref(part)), "templora_sm_partition_create")
    return part


def templora_sm_partition_destroy(part):
    _check(lib.templora_sm_partition_destroy(C.byref(part)), "templora_sm_partition_destroy")


def templora_selftest_bounded_wait(ws, limit_ms=50, stream=None):
    """Enqueue the wait that must run out; read the outcome with templora_read_device_status."""
    _check(lib.templora_selftest_bounded_wait(_ptr(ws), ws.numel(), int(limit_ms), _stream(stream)),
           "templora_selftest_bounded_wait")
