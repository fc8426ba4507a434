"""ctypes binding of libspecverify.so (include/spec_verify.h).

Argument marshalling only: every step of the verify-and-resample pass runs in the CUDA
library.  PyTorch tensors are used as device (or pinned host) buffers and for the
current stream.  If the library has not been built, loading raises -- there is no
fallback of any kind.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# SPECV_LIB names another build of the same library (the debug or the sanitizer build)
LIB_PATH = os.environ.get("SPECV_LIB") or os.path.join(_HERE, "libspecverify.so")

F32, BF16, F16 = 0, 1, 2
ROW_BAD_K, ROW_BAD_TEMPERATURE, ROW_BAD_TOKEN, ROW_ZERO_RESIDUAL = 1, 2, 4, 8
ROW_INTERNAL, ROW_BAD_PARENT = 16, 32

EXPORTS = ("spec_verify", "spec_verify_host", "spec_verify_workspace_bytes",
           "spec_verify_host_arena_bytes", "spec_verify_strerror", "spec_verify_last_cuda_error",
           "spec_verify_launch_count", "spec_verify_set_trace_events", "spec_verify_noalloc", "spec_verify_ex",
           "spec_verify_last_path", "spec_verify_next_lookahead", "spec_verify_selftest_bounded_wait",
           "spec_verify_debug_violation", "spec_verify_from_hidden", "spec_verify_from_hidden_workspace_bytes",
           "spec_verify_from_hidden_status",
           "spec_verify_greedy", "spec_verify_greedy_workspace_bytes",
           "spec_verify_tree", "spec_verify_tree_workspace_bytes")
NOALLOC_SCRATCH_BYTES = 4 << 20

_lib = None


class SpecVerifyError(RuntimeError):
    def __init__(self, status: int, text: str, cuda_error: int = 0):
        super().__init__(f"spec_verify status {status}: {text}" + (f" (cudaError {cuda_error})" if cuda_error else ""))
        self.status = status
        self.cuda_error = cuda_error


def load() -> ctypes.CDLL:
    """dlopen the CUDA library and declare the prototypes of include/spec_verify.h."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2411_00853_b200.build` "
                           "(the CUDA library is the only implementation; there is no fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    common = [vp, vp, ctypes.c_int, i64, i64, i64, vp, vp, i32, i32, i64, vp, ctypes.c_int, vp,
              vp, vp, vp, vp, vp, vp, sz, vp]
    lib.spec_verify.restype = ctypes.c_int
    lib.spec_verify.argtypes = common
    lib.spec_verify_host.restype = ctypes.c_int
    lib.spec_verify_host.argtypes = common + [ctypes.c_uint32]
    lib.spec_verify_noalloc.restype = ctypes.c_int
    lib.spec_verify_noalloc.argtypes = common[:-3] + [vp]
    lib.spec_verify_ex.restype = ctypes.c_int
    lib.spec_verify_ex.argtypes = common + [ctypes.c_uint32, i32, i32, vp]
    lib.spec_verify_next_lookahead.restype = ctypes.c_int
    lib.spec_verify_next_lookahead.argtypes = [vp, i32, vp, i32, i32, i32, vp, vp]
    lib.spec_verify_tree.restype = ctypes.c_int
    lib.spec_verify_tree.argtypes = [vp, vp, ctypes.c_int, i64, i64, i64, vp, vp, vp, i32, i32, i64, vp, ctypes.c_int,
                                     vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, ctypes.c_uint32]
    lib.spec_verify_tree_workspace_bytes.restype = sz
    lib.spec_verify_tree_workspace_bytes.argtypes = [i32, i64, i64]
    lib.spec_verify_greedy.restype = ctypes.c_int
    lib.spec_verify_greedy.argtypes = [vp, ctypes.c_int, i64, i64, vp, vp, i32, i32, i64, vp, vp, vp, vp, vp, sz, vp,
                                       ctypes.c_uint32]
    lib.spec_verify_greedy_workspace_bytes.restype = sz
    lib.spec_verify_greedy_workspace_bytes.argtypes = [i32, i64]
    lib.spec_verify_selftest_bounded_wait.restype = ctypes.c_int
    lib.spec_verify_selftest_bounded_wait.argtypes = [i64, vp, vp]
    lib.spec_verify_last_path.restype = ctypes.c_int
    lib.spec_verify_last_path.argtypes = []
    lib.spec_verify_from_hidden_workspace_bytes.restype = sz
    lib.spec_verify_from_hidden_workspace_bytes.argtypes = [i32, i64, i64]
    lib.spec_verify_from_hidden.restype = ctypes.c_int
    lib.spec_verify_from_hidden.argtypes = [vp, i64, i64, vp, i64, vp, i64, i64, vp, i64, i64, vp, i64, vp, i64, vp, vp, i32,
                                            i32, i64, vp, ctypes.c_int, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.spec_verify_from_hidden_status.restype = ctypes.c_int
    lib.spec_verify_from_hidden_status.argtypes = [vp, i32, i64, i64, vp]
    lib.spec_verify_debug_violation.restype = ctypes.c_int
    lib.spec_verify_debug_violation.argtypes = []
    lib.spec_verify_workspace_bytes.restype = sz
    lib.spec_verify_workspace_bytes.argtypes = [i32, i64, i64]
    lib.spec_verify_host_arena_bytes.restype = sz
    lib.spec_verify_host_arena_bytes.argtypes = [ctypes.c_int, i32, i64, i64]
    lib.spec_verify_strerror.restype = ctypes.c_char_p
    lib.spec_verify_strerror.argtypes = [ctypes.c_int]
    lib.spec_verify_last_cuda_error.restype = ctypes.c_int
    lib.spec_verify_last_cuda_error.argtypes = []
    lib.spec_verify_launch_count.restype = ctypes.c_uint64
    lib.spec_verify_launch_count.argtypes = []
    lib.spec_verify_set_trace_events.restype = ctypes.c_int
    lib.spec_verify_set_trace_events.argtypes = [ctypes.POINTER(ctypes.c_void_p)]
    _lib = lib
    return lib


def _check(rc: int):
    if rc != 0:
        lib = load()
        raise SpecVerifyError(rc, lib.spec_verify_strerror(rc).decode(), lib.spec_verify_last_cuda_error())


def strerror(status: int) -> str:
    return load().spec_verify_strerror(status).decode()


def launch_count() -> int:
    return int(load().spec_verify_launch_count())


def set_trace_events(events):
    """events: four recorded torch.cuda.Event(enable_timing=True), or None to switch tracing off."""
    lib = load()
    if events is None:
        lib.spec_verify_set_trace_events(None)
        return
    arr = (ctypes.c_void_p * 4)(*[ctypes.c_void_p(e.cuda_event) for e in events])
    lib.spec_verify_set_trace_events(arr)


PATH_AUTO, PATH_STREAMING, PATH_RING, PATH_CLUSTER = 0, 1, 2, 3
FLAG_STREAMING, FLAG_RING, FLAG_EARLY_EXIT, FLAG_CLUSTER = 1, 2, 4, 8
_PATH_FLAG = {PATH_AUTO: 0, PATH_STREAMING: FLAG_STREAMING, PATH_RING: FLAG_RING, PATH_CLUSTER: FLAG_CLUSTER}

# The C library keeps no mode between calls: options travel with every call as `flags`.  For
# convenience (tests, the benchmark) this module holds DEFAULT flags that its wrappers pass when
# the caller gives none; they are plain Python state of this module, not of the library.
_default_flags = 0


def set_path(path: int):
    """Default kernel set of this module's wrappers: PATH_AUTO, PATH_STREAMING, PATH_RING or PATH_CLUSTER."""
    global _default_flags
    if path not in _PATH_FLAG:
        raise ValueError("path must be PATH_AUTO, PATH_STREAMING, PATH_RING or PATH_CLUSTER")
    _default_flags = (_default_flags & ~(FLAG_STREAMING | FLAG_RING | FLAG_CLUSTER)) | _PATH_FLAG[path]


def set_early_exit(enable: bool):
    """Default of this module's spec_verify wrapper: skip logits rows after a sequence's first
    clear rejection (ring kernels only; same tokens)."""
    global _default_flags
    _default_flags = (_default_flags | FLAG_EARLY_EXIT) if enable else (_default_flags & ~FLAG_EARLY_EXIT)


def default_flags() -> int:
    return _default_flags


def next_lookahead(k_per_row, accepted_len, k_min: int, k_max: int, *, k_uniform: int = 0, out=None, stream=None):
    """Next round's lookahead per sequence (CUDA int32 tensors): K+2 after a fully accepted draft,
    else K-1, clamped to [k_min, k_max]."""
    B = accepted_len.shape[0]
    if out is None:
        out = torch.empty(B, dtype=torch.int32, device=accepted_len.device)
    if stream is None:
        stream = torch.cuda.current_stream(accepted_len.device).cuda_stream
    _check(load().spec_verify_next_lookahead(_ptr(k_per_row), int(k_uniform), _ptr(accepted_len), B, int(k_min),
                                             int(k_max), _ptr(out), ctypes.c_void_p(stream)))
    return out


def selftest_bounded_wait(limit_cycles: int, stream=None):
    """Runs the library's bounded wait into its limit on purpose (see the header).  Returns
    (error_word, cycles_first_wait, cycles_second_wait, reached_end) as Python ints."""
    out = torch.zeros(4, dtype=torch.int64, device="cuda")
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    _check(load().spec_verify_selftest_bounded_wait(int(limit_cycles), _ptr(out), ctypes.c_void_p(stream)))
    torch.cuda.synchronize()
    return tuple(int(v) for v in out.cpu())


def debug_violation() -> int:
    """Largest range-check site code recorded by a -DSPECV_DEBUG build (0: none; -1: not such a build)."""
    return int(load().spec_verify_debug_violation())


def last_path() -> int:
    return int(load().spec_verify_last_path())


def workspace_bytes(B: int, n_draft_total: int, V: int) -> int:
    return int(load().spec_verify_workspace_bytes(B, n_draft_total, V))


def host_arena_bytes(dtype: int, B: int, n_draft_total: int, V: int) -> int:
    return int(load().spec_verify_host_arena_bytes(dtype, B, n_draft_total, V))


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float16:
        return F16
    raise TypeError("logits must be float32, bfloat16 or float16")


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _temporary_workspace(nbytes: int, dev, stream):
    """Scratch allocated for one call.  When the call runs on a caller-given raw stream, torch's
    allocator is told that the block is in use there, so it is not handed out again before the
    pass has finished."""
    ws = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=dev)
    if stream is not None:
        ws.record_stream(torch.cuda.ExternalStream(int(stream), device=dev))
    return ws


def _shape_args(target_logits, draft_logits, k_per_row, k_uniform):
    assert target_logits.dim() == 2 and target_logits.stride(1) == 1
    V = target_logits.shape[1]
    D = 0 if draft_logits is None else draft_logits.shape[0]
    if k_per_row is None:
        B = target_logits.shape[0] - D
        k_uniform = (D // B if B > 0 else 0) if k_uniform is None else k_uniform
    else:
        B = k_per_row.shape[0]
        k_uniform = 0
    ld_t = target_logits.stride(0) if target_logits.shape[0] > 1 else max(V, target_logits.stride(0))
    if D > 0:
        assert draft_logits.dim() == 2 and draft_logits.stride(1) == 1 and draft_logits.shape[1] == V
        ld_d = draft_logits.stride(0) if D > 1 else max(V, draft_logits.stride(0))
    else:
        ld_d = V
    return V, D, B, int(k_uniform), ld_t, ld_d


def spec_verify(target_logits, draft_logits, draft_tokens, k_per_row, temperature, uniforms, *,
                k_uniform=None, accepted_len=None, emitted_tokens=None, row_status=None,
                diag_p_tok=None, diag_q_tok=None, workspace=None, stream=None, flags=None,
                next_k=None, k_min=0, k_max=0):
    """Enqueue one verify-and-resample pass on CUDA tensors (spec_verify_ex of include/spec_verify.h).

    target_logits [sum(K)+B, V], draft_logits [sum(K), V]: float32 or bfloat16, row pitch = stride(0)
    draft_tokens int32 [sum(K)], k_per_row int32 [B] or None (then every sequence has k_uniform drafts)
    temperature float32 [1] or [B], uniforms float32 [sum(K)+B]
    Returns (accepted_len int32 [B], emitted_tokens int32 [sum(K)+B]); the call is asynchronous
    on `stream` (default: torch's current stream).  Output / scratch tensors may be passed in to
    avoid allocations.  flags: FLAG_* bits (default: this module's default flags); next_k: int32 [B]
    CUDA tensor that receives the next round's lookahead, clamped to [k_min, k_max].
    With a `stream` other than torch's current one, pass a `workspace` you own: a temporary
    allocated here would be returned to torch's allocator while the pass may still be running.
    """
    lib = load()
    dev = target_logits.device
    V, D, B, k_uniform, ld_t, ld_d = _shape_args(target_logits, draft_logits, k_per_row, k_uniform)
    per_row = int(temperature.numel() == B and B > 1)
    if accepted_len is None:
        accepted_len = torch.empty(B, dtype=torch.int32, device=dev)
    if emitted_tokens is None:
        emitted_tokens = torch.empty(D + B, dtype=torch.int32, device=dev)
    need = workspace_bytes(B, D, V)
    if workspace is None:
        workspace = _temporary_workspace(need, dev, stream)
    if stream is None:
        stream = torch.cuda.current_stream(dev).cuda_stream
    rc = lib.spec_verify_ex(_ptr(target_logits), _ptr(draft_logits) if D else None, _dtype_code(target_logits),
                            V, ld_t, ld_d, _ptr(draft_tokens) if D else None, _ptr(k_per_row), B, k_uniform, D,
                            _ptr(temperature), per_row, _ptr(uniforms), _ptr(accepted_len), _ptr(emitted_tokens),
                            _ptr(row_status), _ptr(diag_p_tok), _ptr(diag_q_tok), _ptr(workspace),
                            workspace.numel() * workspace.element_size(), ctypes.c_void_p(stream),
                            _default_flags if flags is None else int(flags), int(k_min), int(k_max), _ptr(next_k))
    _check(rc)
    return accepted_len, emitted_tokens


def spec_verify_noalloc(target_logits, draft_logits, draft_tokens, k_per_row, temperature, uniforms,
                        accepted_len, emitted_tokens, *, k_uniform=None, row_status=None,
                        diag_p_tok=None, diag_q_tok=None, stream=None):
    """spec_verify without a workspace argument, for callers that may not allocate device
    memory: the library's built-in static scratch (NOALLOC_SCRATCH_BYTES) is used instead.
    This wrapper allocates nothing either, so the output tensors are required arguments.
    Calls share that scratch: keep them on one stream (or otherwise serialised)."""
    lib = load()
    V, D, B, k_uniform, ld_t, ld_d = _shape_args(target_logits, draft_logits, k_per_row, k_uniform)
    per_row = int(temperature.numel() == B and B > 1)
    if stream is None:
        stream = torch.cuda.current_stream(target_logits.device).cuda_stream
    rc = lib.spec_verify_noalloc(_ptr(target_logits), _ptr(draft_logits) if D else None,
                                 _dtype_code(target_logits), V, ld_t, ld_d, _ptr(draft_tokens) if D else None,
                                 _ptr(k_per_row), B, k_uniform, D, _ptr(temperature), per_row, _ptr(uniforms),
                                 _ptr(accepted_len), _ptr(emitted_tokens), _ptr(row_status), _ptr(diag_p_tok),
                                 _ptr(diag_q_tok), ctypes.c_void_p(stream))
    _check(rc)
    return accepted_len, emitted_tokens


def spec_verify_host(target_logits, draft_logits, draft_tokens, k_per_row, temperature, uniforms, arena, *,
                     k_uniform=None, accepted_len=None, emitted_tokens=None, row_status=None,
                     diag_p_tok=None, diag_q_tok=None, stream=None, flags=None):
    """The same pass on HOST tensors (CPU torch tensors, ideally pinned); `arena` is a CUDA uint8
    tensor of at least host_arena_bytes(...) bytes.  Blocks until the outputs are on the host."""
    lib = load()
    V, D, B, k_uniform, ld_t, ld_d = _shape_args(target_logits, draft_logits, k_per_row, k_uniform)
    per_row = int(temperature.numel() == B and B > 1)
    if accepted_len is None:
        accepted_len = torch.empty(B, dtype=torch.int32).pin_memory()
    if emitted_tokens is None:
        emitted_tokens = torch.empty(D + B, dtype=torch.int32).pin_memory()
    if stream is None:
        stream = torch.cuda.current_stream(arena.device).cuda_stream
    rc = lib.spec_verify_host(_ptr(target_logits), _ptr(draft_logits) if D else None, _dtype_code(target_logits),
                              V, ld_t, ld_d, _ptr(draft_tokens) if D else None, _ptr(k_per_row), B, k_uniform, D,
                              _ptr(temperature), per_row, _ptr(uniforms), _ptr(accepted_len), _ptr(emitted_tokens),
                              _ptr(row_status), _ptr(diag_p_tok), _ptr(diag_q_tok), _ptr(arena),
                              arena.numel() * arena.element_size(), ctypes.c_void_p(stream),
                              _default_flags if flags is None else int(flags))
    _check(rc)
    return accepted_len, emitted_tokens


def _path_flags(flags) -> int:
    """Flags for the entry points that take a kernel-set choice only."""
    return (_default_flags if flags is None else int(flags)) & (FLAG_STREAMING | FLAG_RING)


def greedy_workspace_bytes(B: int, n_draft_total: int) -> int:
    return int(load().spec_verify_greedy_workspace_bytes(B, n_draft_total))


def spec_verify_greedy(target_logits, draft_tokens, k_per_row, *, k_uniform=None, accepted_len=None,
                       emitted_tokens=None, row_status=None, target_argmax=None, workspace=None, stream=None,
                       flags=None):
    """Enqueue one greedy verification pass (temperature -> 0: accept while the draft token is the
    target row's argmax) on CUDA tensors.  target_logits [sum(K)+B, V]; draft_tokens int32 [sum(K)];
    k_per_row int32 [B] or None with k_uniform.  Returns (accepted_len, emitted_tokens)."""
    lib = load()
    dev = target_logits.device
    assert target_logits.dim() == 2 and target_logits.stride(1) == 1
    V = target_logits.shape[1]
    if k_per_row is None:
        assert k_uniform is not None
        B = target_logits.shape[0] // (int(k_uniform) + 1)
    else:
        B, k_uniform = k_per_row.shape[0], 0
    D = target_logits.shape[0] - B
    ld_t = target_logits.stride(0) if target_logits.shape[0] > 1 else max(V, target_logits.stride(0))
    if accepted_len is None:
        accepted_len = torch.empty(B, dtype=torch.int32, device=dev)
    if emitted_tokens is None:
        emitted_tokens = torch.empty(D + B, dtype=torch.int32, device=dev)
    if workspace is None:
        workspace = _temporary_workspace(greedy_workspace_bytes(B, D), dev, stream)
    if stream is None:
        stream = torch.cuda.current_stream(dev).cuda_stream
    rc = lib.spec_verify_greedy(_ptr(target_logits), _dtype_code(target_logits), V, ld_t,
                                _ptr(draft_tokens) if D else None, _ptr(k_per_row), B, int(k_uniform), D,
                                _ptr(accepted_len), _ptr(emitted_tokens), _ptr(row_status), _ptr(target_argmax),
                                _ptr(workspace), workspace.numel() * workspace.element_size(),
                                ctypes.c_void_p(stream), _path_flags(flags))
    _check(rc)
    return accepted_len, emitted_tokens


def tree_workspace_bytes(B: int, n_node_total: int, V: int) -> int:
    return int(load().spec_verify_tree_workspace_bytes(B, n_node_total, V))


def spec_verify_tree(target_logits, draft_logits, node_tokens, node_parent, n_per_seq, temperature, uniforms, *,
                     n_uniform=None, accepted_len=None, emitted_tokens=None, accepted_nodes=None, row_status=None,
                     diag_p_tok=None, diag_q_tok=None, workspace=None, stream=None, flags=None):
    """Enqueue one tree-structured verification pass on CUDA tensors (see include/spec_verify.h).
    target_logits [sum(N)+B, V] (row of context c), draft_logits [sum(N), V], node_tokens / node_parent
    int32 [sum(N)], n_per_seq int32 [B] (or None with n_uniform).  Returns (accepted_len, emitted_tokens)."""
    lib = load()
    dev = target_logits.device
    V, D, B, n_uniform, ld_t, ld_d = _shape_args(target_logits, draft_logits, n_per_seq, n_uniform)
    per_seq = int(temperature.numel() == B and B > 1)
    if accepted_len is None:
        accepted_len = torch.empty(B, dtype=torch.int32, device=dev)
    if emitted_tokens is None:
        emitted_tokens = torch.empty(D + B, dtype=torch.int32, device=dev)
    if workspace is None:
        workspace = _temporary_workspace(tree_workspace_bytes(B, D, V), dev, stream)
    if stream is None:
        stream = torch.cuda.current_stream(dev).cuda_stream
    rc = lib.spec_verify_tree(_ptr(target_logits), _ptr(draft_logits) if D else None, _dtype_code(target_logits),
                              V, ld_t, ld_d, _ptr(node_tokens) if D else None, _ptr(node_parent) if D else None,
                              _ptr(n_per_seq), B, n_uniform, D, _ptr(temperature), per_seq, _ptr(uniforms),
                              _ptr(accepted_len), _ptr(emitted_tokens), _ptr(accepted_nodes), _ptr(row_status),
                              _ptr(diag_p_tok), _ptr(diag_q_tok), _ptr(workspace),
                              workspace.numel() * workspace.element_size(), ctypes.c_void_p(stream),
                              _path_flags(flags))
    _check(rc)
    return accepted_len, emitted_tokens


def from_hidden_workspace_bytes(B: int, n_draft_total: int, V: int) -> int:
    return int(load().spec_verify_from_hidden_workspace_bytes(B, n_draft_total, V))


def spec_verify_from_hidden(target_hidden, target_weight, draft_hidden, draft_weight, draft_tokens, k_per_row,
                            temperature, uniforms, *, k_uniform=None, target_logits=None, draft_logits=None,
                            accepted_len=None, emitted_tokens=None, row_status=None, diag_p_tok=None,
                            diag_q_tok=None, workspace=None, stream=None):
    """The verify pass from hidden states (bf16 CUDA tensors): target_hidden [sum(K)+B, H], target_weight
    [V, H], draft_hidden [sum(K), Hd], draft_weight [V, Hd].  The logits (bf16) are written to
    target_logits / draft_logits.  Returns (accepted_len, emitted_tokens, target_logits, draft_logits)."""
    lib = load()
    dev = target_hidden.device
    V = target_weight.shape[0]
    D = 0 if draft_hidden is None else draft_hidden.shape[0]
    if k_per_row is None:
        B = target_hidden.shape[0] - D
        k_uniform = (D // B if B > 0 else 0) if k_uniform is None else k_uniform
    else:
        B, k_uniform = k_per_row.shape[0], 0
    if target_logits is None:
        target_logits = torch.empty((D + B, V), dtype=torch.bfloat16, device=dev)
    if draft_logits is None:
        draft_logits = torch.empty((max(D, 1), V), dtype=torch.bfloat16, device=dev)[:D]
    if accepted_len is None:
        accepted_len = torch.empty(B, dtype=torch.int32, device=dev)
    if emitted_tokens is None:
        emitted_tokens = torch.empty(D + B, dtype=torch.int32, device=dev)
    if workspace is None:
        workspace = _temporary_workspace(from_hidden_workspace_bytes(B, D, V), dev, stream)
    if stream is None:
        stream = torch.cuda.current_stream(dev).cuda_stream
    per_row = int(temperature.numel() == B and B > 1)
    ld = lambda t: t.stride(0) if t.shape[0] > 1 else max(t.shape[1], t.stride(0))
    rc = lib.spec_verify_from_hidden(
        _ptr(target_hidden), ld(target_hidden), target_hidden.shape[1], _ptr(target_weight), ld(target_weight),
        _ptr(draft_hidden) if D else None, ld(draft_hidden) if D else 0, draft_hidden.shape[1] if D else 0,
        _ptr(draft_weight) if D else None, ld(draft_weight) if D else 0, V,
        _ptr(target_logits), ld(target_logits), _ptr(draft_logits) if D else None, ld(draft_logits) if D else V,
        _ptr(draft_tokens) if D else None, _ptr(k_per_row), B, int(k_uniform), D, _ptr(temperature), per_row,
        _ptr(uniforms), _ptr(accepted_len), _ptr(emitted_tokens), _ptr(row_status), _ptr(diag_p_tok), _ptr(diag_q_tok),
        _ptr(workspace), workspace.numel() * workspace.element_size(), ctypes.c_void_p(stream))
    _check(rc)
    return accepted_len, emitted_tokens, target_logits, draft_logits


def from_hidden_status(workspace, B: int, n_draft_total: int, V: int, stream=None) -> int:
    if stream is None:
        stream = torch.cuda.current_stream(workspace.device).cuda_stream
    return int(load().spec_verify_from_hidden_status(_ptr(workspace), B, n_draft_total, V, ctypes.c_void_p(stream)))
