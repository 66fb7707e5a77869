"""ctypes binding of the C-ABI library declared in include/fdd.h.

Argument marshalling only: every function below has the name and the argument
order of its C counterpart, takes torch CUDA tensors (or raw integer device
pointers) where the C call takes device pointers, and raises `FddError` when the
C call returns a negative status.  All arithmetic runs in the CUDA kernels of
libfdd.so; there is no fallback, and a missing library is an error.
"""
import ctypes
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libfdd.so")

FDD_OK = 0
FDD_ERR_INVALID_ARG, FDD_ERR_SHAPE, FDD_ERR_CAPACITY, FDD_ERR_STATE = -1, -2, -3, -4
FDD_ERR_CUDA, FDD_ERR_DEVICE_TIMEOUT, FDD_ERR_UNSUPPORTED = -5, -6, -7
FDD_MASKED, FDD_COMMITTED, FDD_SCAFFOLD, FDD_DRAFT = 0, 1, 2, 3
FDD_LOGITS_F32, FDD_LOGITS_BF16 = 0, 1

EXPORTS = (
    "fdd_create", "fdd_destroy", "fdd_last_error", "fdd_launch_count", "fdd_fork",
    "fdd_forkset_free", "fdd_forkset_suffix_len", "fdd_forkset_reset", "fdd_block_attn", "fdd_block_attn_gated", "fdd_average_rollouts_jmt", "fdd_unmask_counted",
    "fdd_unmask", "fdd_ss_draft", "fdd_ss_accept", "fdd_kv_commit", "fdd_average_rollouts", "fdd_poll_status", "fdd_unmask_static", "fdd_plan_blocks", "fdd_upload_masked_rows",
    "fdd_prefix_extend", "fdd_forkset_prefix_len", "fdd_set_merge_wait_limit", "fdd_decode_block", "fdd_pull_masked_rows",
)
FDD_UNMASK_STATIC_MAX_RECORDS = 65536


class FddError(RuntimeError):
    def __init__(self, status, text):
        super().__init__(f"fdd status {status}: {text}")
        self.status = status


class fdd_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in (
        "n_q_heads", "n_kv_heads", "head_dim", "vocab", "n_layers", "page_tokens",
        "max_block", "max_forks", "logits_dtype")]


_lib_handle = None


def lib():
    """The loaded shared library.  Raises if it has not been built."""
    global _lib_handle
    if _lib_handle is not None:
        return _lib_handle
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2605_23163_b200.build` "
            "(there is no CPU fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, ip, i32, u32, u64, f32 = (ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32), ctypes.c_int,
                                  ctypes.c_uint32, ctypes.c_uint64, ctypes.c_float)
    vpp = ctypes.POINTER(ctypes.c_void_p)
    L.fdd_create.argtypes = [ctypes.POINTER(fdd_config), vpp]
    L.fdd_create.restype = i32
    L.fdd_destroy.argtypes = [vp]
    L.fdd_destroy.restype = None
    L.fdd_last_error.argtypes = [vp]
    L.fdd_last_error.restype = ctypes.c_char_p
    L.fdd_launch_count.argtypes = [vp]
    L.fdd_launch_count.restype = u64
    L.fdd_fork.argtypes = [vp, vpp, vpp, vp, i32, i32, i32, ctypes.POINTER(u64), vpp, vpp, i32, vpp]
    L.fdd_fork.restype = i32
    L.fdd_forkset_free.argtypes = [vp, vp]
    L.fdd_forkset_free.restype = i32
    L.fdd_forkset_suffix_len.argtypes = [vp]
    L.fdd_forkset_suffix_len.restype = i32
    L.fdd_forkset_reset.argtypes = [vp, vp]
    L.fdd_forkset_reset.restype = i32
    L.fdd_block_attn.argtypes = [vp, vpp, i32, i32, vp, vp, vp, vp, ip, f32, i32, vp]
    L.fdd_block_attn.restype = i32
    L.fdd_block_attn_gated.argtypes = [vp, vpp, i32, i32, vp, vp, vp, vp, ip, f32, i32, vp, vp]
    L.fdd_block_attn_gated.restype = i32
    L.fdd_unmask.argtypes = [vp, vpp, i32, vp, vp, vp, ip, f32, f32, u32, u32, vp, vp, vp, vp]
    L.fdd_unmask.restype = i32
    L.fdd_unmask_counted.argtypes = [vp, vpp, i32, vp, vp, vp, ip, f32, f32, u32, vp, vp, vp, vp, vp]
    L.fdd_unmask_counted.restype = i32
    for fn in (L.fdd_ss_draft, L.fdd_ss_accept):
        fn.argtypes = [vp, vpp, i32, vp, vp, vp, ip, f32, u32, u32, vp, vp, vp]
        fn.restype = i32
    L.fdd_kv_commit.argtypes = [vp, vpp, i32, i32, vp, vp, ip, i32, vp]
    L.fdd_kv_commit.restype = i32
    L.fdd_prefix_extend.argtypes = [vp, vpp, i32, i32, vp, vp, ip, i32, vp]
    L.fdd_prefix_extend.restype = i32
    L.fdd_forkset_prefix_len.argtypes = [vp]
    L.fdd_forkset_prefix_len.restype = i32
    L.fdd_set_merge_wait_limit.argtypes = [vp, ctypes.c_longlong]
    L.fdd_set_merge_wait_limit.restype = i32
    L.fdd_average_rollouts.argtypes = [vp, vp, i32, i32, vp, vp]
    L.fdd_average_rollouts.restype = i32
    L.fdd_average_rollouts_jmt.argtypes = [vp, vp, i32, i32, i32, vp, vp]
    L.fdd_average_rollouts_jmt.restype = i32
    L.fdd_poll_status.argtypes = [vp, vp]
    L.fdd_poll_status.restype = i32
    L.fdd_unmask_static.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, f32, f32, u32, u32, vp, vp, vp, vp,
                                    ctypes.c_char_p, ctypes.c_size_t]
    L.fdd_unmask_static.restype = i32
    L.fdd_decode_block.argtypes = [vp, vpp, i32, i32, i32, i32, vpp, vpp, vpp, vpp, vpp, vp, vp, ip, f32, i32, f32, f32, u32,
                                   i32, vp, vp, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int), vp, vp, vp]
    L.fdd_decode_block.restype = i32
    _lib_handle = L
    return L


def _ptr(t):
    """Device address of a tensor (must be contiguous) or a raw integer pointer / None."""
    if t is None:
        return None
    if isinstance(t, ctypes.c_void_p):
        return t
    if isinstance(t, int):
        return ctypes.c_void_p(t)
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if isinstance(stream, ctypes.c_void_p):
        return stream
    if stream is None:
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return ctypes.c_void_p(stream)
    return ctypes.c_void_p(stream.cuda_stream)


def _check(ctx, status):
    if status < 0:
        raise FddError(status, lib().fdd_last_error(ctx).decode() if ctx else "no context")
    return status


def _ptr_array(items):
    if isinstance(items, ctypes.Array):      # marshalled earlier by ptr_array()
        return items
    arr = (ctypes.c_void_p * len(items))()
    for i, t in enumerate(items):
        p = _ptr(t)
        arr[i] = p.value if p is not None else None
    return arr


def _i32_array(vals):
    if isinstance(vals, ctypes.Array):       # marshalled earlier by i32_array()
        return vals
    return (ctypes.c_int32 * len(vals))(*[int(v) for v in vals])


def ptr_array(items):
    """Marshal a list of tensors / handles once; the result can be passed wherever the binding
    takes such a list (saves the conversion in a loop that passes the same list every step)."""
    return _ptr_array(items)


def i32_array(vals):
    """Marshal a list of ints once (see ptr_array)."""
    return _i32_array(vals)


def u64_array(vals):
    """Marshal a list of 64-bit seeds once (see ptr_array)."""
    vals = [int(s) & 0xFFFFFFFFFFFFFFFF for s in vals]
    return (ctypes.c_uint64 * len(vals))(*vals)


def fdd_create(n_q_heads, n_kv_heads, head_dim, vocab, n_layers=1, page_tokens=0, max_block=64,
               max_forks=32, logits_dtype=FDD_LOGITS_BF16):
    cfg = fdd_config(n_q_heads, n_kv_heads, head_dim, vocab, n_layers, page_tokens, max_block,
                     max_forks, logits_dtype)
    out = ctypes.c_void_p()
    st = lib().fdd_create(ctypes.byref(cfg), ctypes.byref(out))
    if st < 0:
        raise FddError(st, "fdd_create failed")
    return out


def fdd_destroy(ctx):
    lib().fdd_destroy(ctx)


def fdd_last_error(ctx):
    return lib().fdd_last_error(ctx).decode()


def fdd_launch_count(ctx):
    return int(lib().fdd_launch_count(ctx))


def fdd_fork(ctx, prefix_k, prefix_v, page_table, prefix_len, prefix_capacity, n_forks, seeds,
             suffix_k, suffix_v, suffix_capacity):
    """prefix_k/v, suffix_k/v: per-layer lists of CUDA tensors; seeds: iterable of N ints."""
    seed_arr = seeds if isinstance(seeds, ctypes.Array) else u64_array(seeds)
    out = ctypes.c_void_p()
    st = lib().fdd_fork(ctx, _ptr_array(prefix_k), _ptr_array(prefix_v), _ptr(page_table),
                        int(prefix_len), int(prefix_capacity), int(n_forks), seed_arr,
                        _ptr_array(suffix_k), _ptr_array(suffix_v), int(suffix_capacity),
                        ctypes.byref(out))
    _check(ctx, st)
    return out


def fdd_forkset_free(ctx, fs):
    return _check(ctx, lib().fdd_forkset_free(ctx, fs))


def fdd_forkset_suffix_len(fs):
    return int(lib().fdd_forkset_suffix_len(fs))


def fdd_forkset_reset(ctx, fs):
    return _check(ctx, lib().fdd_forkset_reset(ctx, fs))


def fdd_block_attn(ctx, sets, layer, q, k_blk, v_blk, out, block_len, scale, causal_in_block=0,
                   stream=None):
    return _check(ctx, lib().fdd_block_attn(
        ctx, _ptr_array(sets), len(sets), int(layer), _ptr(q), _ptr(k_blk), _ptr(v_blk), _ptr(out),
        _i32_array(block_len), float(scale), int(causal_in_block), _stream(stream)))


def fdd_block_attn_gated(ctx, sets, layer, q, k_blk, v_blk, out, block_len, scale, causal_in_block, gate,
                         stream=None):
    return _check(ctx, lib().fdd_block_attn_gated(
        ctx, _ptr_array(sets), len(sets), int(layer), _ptr(q), _ptr(k_blk), _ptr(v_blk), _ptr(out),
        _i32_array(block_len), float(scale), int(causal_in_block), _ptr(gate), _stream(stream)))


def fdd_unmask(ctx, sets, logits, tokens, state, block_len, threshold, temperature, block_idx, step,
               n_committed, n_left, conf=None, stream=None):
    return _check(ctx, lib().fdd_unmask(
        ctx, _ptr_array(sets), len(sets), _ptr(logits), _ptr(tokens), _ptr(state),
        _i32_array(block_len), float(threshold), float(temperature), int(block_idx), int(step),
        _ptr(n_committed), _ptr(n_left), _ptr(conf), _stream(stream)))


def fdd_decode_block(ctx, sets, n_layers, max_steps, q, k_blk, v_blk, out, logits, tokens, state, block_len, scale,
                     causal_in_block, threshold, temperature, block_idx, commit_kv, n_committed, n_left, stream=None):
    """The denoising loop of one block, run by the library.  q, k_blk, v_blk, out: per resident input
    set a list of n_layers tensors (or arrays made by ptr_array over the flattened [set][layer] list);
    logits: one tensor per input set.  Returns (steps_taken, masked_left)."""
    n_inputs = len(logits)

    def flat(x):
        return x if isinstance(x, ctypes.Array) else _ptr_array([t for per_set in x for t in per_set])

    steps, left = ctypes.c_int(0), ctypes.c_int(0)
    _check(ctx, lib().fdd_decode_block(
        ctx, _ptr_array(sets), len(sets), int(n_layers), int(max_steps), int(n_inputs),
        flat(q), flat(k_blk), flat(v_blk), flat(out), _ptr_array(logits), _ptr(tokens), _ptr(state),
        _i32_array(block_len), float(scale), int(causal_in_block), float(threshold), float(temperature),
        int(block_idx), int(commit_kv), _ptr(n_committed), _ptr(n_left), ctypes.byref(steps), ctypes.byref(left),
        None, None, _stream(stream)))
    return steps.value, left.value


def decode_block_call(ctx, sets, n_layers, max_steps, q, k_blk, v_blk, out, logits, tokens, state, block_len, scale,
                      causal_in_block, threshold, temperature, block_idx, commit_kv, n_committed, n_left, stream=None):
    """The arguments of fdd_decode_block marshalled once: returns call() -> (steps_taken, masked_left) for a
    caller that repeats the same call block after block (the conversion costs more than a short block's
    first launch)."""
    n_inputs = len(logits)

    def flat(x):
        return x if isinstance(x, ctypes.Array) else _ptr_array([t for per_set in x for t in per_set])

    steps, left = ctypes.c_int(0), ctypes.c_int(0)
    fn = lib().fdd_decode_block
    args = (ctx, _ptr_array(sets), len(sets), int(n_layers), int(max_steps), int(n_inputs),
            flat(q), flat(k_blk), flat(v_blk), flat(out), _ptr_array(logits), _ptr(tokens), _ptr(state),
            _i32_array(block_len), float(scale), int(causal_in_block), float(threshold), float(temperature),
            int(block_idx), int(commit_kv), _ptr(n_committed), _ptr(n_left), ctypes.byref(steps), ctypes.byref(left),
            None, None, _stream(stream))

    def call():
        status = fn(*args)
        if status < 0:
            _check(ctx, status)
        return steps.value, left.value

    return call


def fdd_unmask_counted(ctx, sets, logits, tokens, state, block_len, threshold, temperature, block_idx,
                       step_counter, n_committed, n_left, conf=None, stream=None):
    return _check(ctx, lib().fdd_unmask_counted(
        ctx, _ptr_array(sets), len(sets), _ptr(logits), _ptr(tokens), _ptr(state),
        _i32_array(block_len), float(threshold), float(temperature), int(block_idx), _ptr(step_counter),
        _ptr(n_committed), _ptr(n_left), _ptr(conf), _stream(stream)))


def fdd_ss_draft(ctx, sets, logits, tokens, state, block_len, temperature, block_idx, step, n_drafted, n_left,
                 stream=None):
    return _check(ctx, lib().fdd_ss_draft(
        ctx, _ptr_array(sets), len(sets), _ptr(logits), _ptr(tokens), _ptr(state), _i32_array(block_len),
        float(temperature), int(block_idx), int(step), _ptr(n_drafted), _ptr(n_left), _stream(stream)))


def fdd_ss_accept(ctx, sets, ar_logits, tokens, state, block_len, temperature, block_idx, step, n_accepted, n_left,
                  stream=None):
    return _check(ctx, lib().fdd_ss_accept(
        ctx, _ptr_array(sets), len(sets), _ptr(ar_logits), _ptr(tokens), _ptr(state), _i32_array(block_len),
        float(temperature), int(block_idx), int(step), _ptr(n_accepted), _ptr(n_left), _stream(stream)))


def fdd_kv_commit(ctx, sets, layer, k_blk, v_blk, block_len, advance, stream=None):
    return _check(ctx, lib().fdd_kv_commit(
        ctx, _ptr_array(sets), len(sets), int(layer), _ptr(k_blk), _ptr(v_blk),
        _i32_array(block_len), int(advance), _stream(stream)))


def fdd_prefix_extend(ctx, sets, layer, k_blk, v_blk, block_len, advance, stream=None):
    return _check(ctx, lib().fdd_prefix_extend(
        ctx, _ptr_array(sets), len(sets), int(layer), _ptr(k_blk), _ptr(v_blk),
        _i32_array(block_len), int(advance), _stream(stream)))


def fdd_forkset_prefix_len(fs):
    return int(lib().fdd_forkset_prefix_len(fs))


def fdd_set_merge_wait_limit(ctx, sm_clocks):
    return _check(ctx, lib().fdd_set_merge_wait_limit(ctx, int(sm_clocks)))


def fdd_average_rollouts_jmt(ctx, traj, n, w, w_out, out, stream=None):
    return _check(ctx, lib().fdd_average_rollouts_jmt(ctx, _ptr(traj), int(n), int(w), int(w_out), _ptr(out),
                                                       _stream(stream)))


def fdd_average_rollouts(ctx, traj, n, w, out, stream=None):
    return _check(ctx, lib().fdd_average_rollouts(ctx, _ptr(traj), int(n), int(w), _ptr(out),
                                                  _stream(stream)))


def average_rollouts_call(ctx, traj, n, w, out, stream=None):
    """The arguments of fdd_average_rollouts marshalled once: returns call() for a caller that repeats it."""
    fn = lib().fdd_average_rollouts
    args = (ctx, _ptr(traj), int(n), int(w), _ptr(out), _stream(stream))

    def call():
        status = fn(*args)
        if status < 0:
            _check(ctx, status)

    return call


def fdd_plan_blocks(editable, section_end, d, capacity=4096):
    """Host-side block planner; returns a list of (begin, end, section)."""
    import numpy as np
    ed = np.ascontiguousarray(editable, dtype=np.uint8)
    en = np.ascontiguousarray(section_end, dtype=np.int32)
    bb, be, bs = (np.zeros(capacity, dtype=np.int32) for _ in range(3))
    n = ctypes.c_int(0)
    L = lib()
    L.fdd_plan_blocks.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                  ctypes.POINTER(ctypes.c_int)]
    L.fdd_plan_blocks.restype = ctypes.c_int
    st = L.fdd_plan_blocks(ed.ctypes.data, en.ctypes.data, len(en), len(ed), int(d), bb.ctypes.data, be.ctypes.data,
                           bs.ctypes.data, capacity, ctypes.byref(n))
    if st < 0:
        raise FddError(st, "fdd_plan_blocks failed")
    return [(int(bb[i]), int(be[i]), int(bs[i])) for i in range(n.value)]


def fdd_pull_masked_rows(ctx, host_logits, dev_logits, dev_state, bytes_pulled=None, stream=None):
    """host_logits: pinned CPU tensor [rows, V]; dev_logits: CUDA tensor of the same shape; dev_state: CUDA
    uint8 tensor [rows]; bytes_pulled: CUDA int64 tensor of one element or None."""
    L = lib()
    L.fdd_pull_masked_rows.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                       ctypes.c_void_p, ctypes.c_void_p]
    L.fdd_pull_masked_rows.restype = ctypes.c_int
    return _check(ctx, L.fdd_pull_masked_rows(ctx, _ptr(host_logits), _ptr(dev_logits), _ptr(dev_state),
                                              int(dev_state.numel()), _ptr(bytes_pulled), _stream(stream)))


def fdd_upload_masked_rows(ctx, host_logits, dev_logits, host_state, stream=None):
    """host_logits: pinned CPU tensor [rows, V]; dev_logits: CUDA tensor of the same shape;
    host_state: CPU uint8 tensor [rows].  Returns the bytes enqueued."""
    L = lib()
    L.fdd_upload_masked_rows.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                         ctypes.POINTER(ctypes.c_size_t), ctypes.c_void_p]
    L.fdd_upload_masked_rows.restype = ctypes.c_int
    n = ctypes.c_size_t(0)
    _check(ctx, L.fdd_upload_masked_rows(ctx, _ptr(host_logits), _ptr(dev_logits), _ptr(host_state),
                                          int(host_state.numel()), ctypes.byref(n), _stream(stream)))
    return int(n.value)


def fdd_poll_status(ctx, stream=None):
    return _check(ctx, lib().fdd_poll_status(ctx, _stream(stream)))


def fdd_unmask_static(logits, logits_dtype, n_forks, block_len, vocab, tokens, state, seeds, threshold,
                      temperature, block_idx, step, n_committed, n_left, conf=None, stream=None):
    """The allocation-free unmasking step: no context, no fork set; `seeds` is a device uint64/int64
    tensor [n_forks].  Raises FddError with the library's message on a negative status."""
    buf = ctypes.create_string_buffer(256)
    st = lib().fdd_unmask_static(_ptr(logits), int(logits_dtype), int(n_forks), int(block_len), int(vocab),
                                 _ptr(tokens), _ptr(state), _ptr(seeds), float(threshold), float(temperature),
                                 int(block_idx), int(step), _ptr(n_committed), _ptr(n_left), _ptr(conf),
                                 _stream(stream), buf, len(buf))
    if st < 0:
        raise FddError(st, buf.value.decode())
    return st
