"""Thin ctypes binding of libstateflow.so: argument marshalling only.

Every function has the name and meaning of the C entry point in include/stateflow.h and takes
torch CUDA tensors for the device pointers.  PyTorch provides device memory and streams; all
arithmetic runs in the library's kernels.  There is no fallback: if the library is missing or a
call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libstateflow.so")
_lib = None

SF_BF16, SF_F32 = 0, 1
STATUS = {0: "SF_OK", 1: "SF_ERR_INVALID_ARG", 2: "SF_ERR_UNSUPPORTED", 3: "SF_ERR_WORKSPACE", 4: "SF_ERR_CUDA",
          5: "SF_ERR_TIMEOUT"}


class SfError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (%s)" % (where, STATUS.get(code, code), status_string(code)))


class SegDesc(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("d_k", ctypes.c_int32), ("d_v", ctypes.c_int32),
                ("seg_len", ctypes.c_int32), ("chunk", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("chunks_per_block", ctypes.c_int32),
                ("tok_stride_qk", ctypes.c_int64), ("tok_stride_v", ctypes.c_int64), ("tok_stride_g", ctypes.c_int64),
                ("batch_stride_qk", ctypes.c_int64), ("batch_stride_v", ctypes.c_int64), ("batch_stride_g", ctypes.c_int64)]


def load() -> ctypes.CDLL:
    """Load the CUDA library; raises if it has not been built (there is no CPU path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libstateflow.so is missing: run `python -m paper_2608_06838_b200.build` "
                               "(or __graft_entry__.build()); this package has no CPU fallback")
        lib = ctypes.CDLL(LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
        dp = ctypes.POINTER(SegDesc)
        ip = ctypes.POINTER(ctypes.c_int32)
        lib.sf_status_string.restype = ctypes.c_char_p
        lib.sf_status_string.argtypes = [ctypes.c_int]
        lib.sf_num_blocks.restype = i32
        lib.sf_num_blocks.argtypes = [dp]
        lib.sf_workspace_bytes.restype = sz
        lib.sf_workspace_bytes.argtypes = [dp, ctypes.c_int]
        lib.sf_segment_fwd.restype = ctypes.c_int
        lib.sf_segment_fwd.argtypes = [dp] + [vp] * 7 + [vp, sz, vp]
        lib.sf_segment_fwd_static.restype = ctypes.c_int
        lib.sf_segment_fwd_static.argtypes = [dp] + [vp] * 7 + [vp]
        lib.sf_segment_bwd.restype = ctypes.c_int
        lib.sf_segment_bwd.argtypes = [dp] + [vp] * 12 + [vp, vp, sz, vp]
        lib.sf_state_scan.restype = ctypes.c_int
        lib.sf_state_scan.argtypes = [dp, i32, i32] + [vp] * 5 + [vp]
        lib.sf_chain_workspace_bytes.restype = sz
        lib.sf_chain_workspace_bytes.argtypes = [dp, ip, i32, ctypes.c_int]
        lib.sf_chain_fwd.restype = ctypes.c_int
        lib.sf_chain_fwd.argtypes = [dp, ip, i32] + [vp] * 7 + [vp, sz, i32, vp]
        lib.sf_chain_bwd.restype = ctypes.c_int
        lib.sf_chain_bwd.argtypes = [dp, ip, i32] + [vp] * 12 + [vp, vp, sz, i32, vp]
        lib.sf_e2e_device_bytes.restype = sz
        lib.sf_e2e_device_bytes.argtypes = [dp, ip, i32]
        lib.sf_chain_fwd_bwd_host.restype = ctypes.c_int
        lib.sf_chain_fwd_bwd_host.argtypes = [dp, ip, i32] + [vp] * 14 + [vp, sz, vp]
        lib.sf_chain_graph_create.restype = ctypes.c_int
        lib.sf_chain_graph_create.argtypes = [dp, ip, i32] + [vp] * 7 + [vp, sz] + [vp] * 7 + [vp, sz, i32, vp,
                                                                                             ctypes.POINTER(vp)]
        lib.sf_chain_graph_launch.restype = ctypes.c_int
        lib.sf_chain_graph_launch.argtypes = [vp, vp]
        lib.sf_chain_graph_kernels.restype = ctypes.c_int64
        lib.sf_chain_graph_kernels.argtypes = [vp]
        lib.sf_chain_graph_destroy.restype = None
        lib.sf_chain_graph_destroy.argtypes = [vp]
        lib.sf_chain_autotune.restype = ctypes.c_int
        lib.sf_chain_autotune.argtypes = [dp, ip, i32] + [vp] * 7 + [vp, sz] + [vp] * 7 + [vp, sz, ip, i32, i32, i32, vp, ip,
                                                                                         ctypes.POINTER(ctypes.c_float)]
        lib.sf_chain_autotune_schedule.restype = ctypes.c_int
        lib.sf_chain_autotune_schedule.argtypes = [dp, ip, i32] + [vp] * 7 + [vp, sz] + [vp] * 7 + [vp, sz, i32, ctypes.c_float, vp,
                                                                                                  vp, vp, vp]
        lib.sf_partition_hybrid.restype = ctypes.c_int
        lib.sf_partition_hybrid.argtypes = [ctypes.c_int64, i32, ctypes.c_double, ctypes.c_double, ctypes.c_double, i32, ip]
        lib.sf_device_status.restype = i32
        lib.sf_device_status_clear.restype = None
        lib.sf_launch_count.restype = ctypes.c_int64
        lib.sf_stage_timing.restype = None
        lib.sf_stage_timing.argtypes = [i32]
        lib.sf_stage_timing_read.restype = i32
        lib.sf_stage_timing_read.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int64), i32]
        lib.sf_recurrent_workspace_bytes.restype = sz
        lib.sf_recurrent_workspace_bytes.argtypes = [dp]
        lib.sf_channel_segment_fwd.restype = ctypes.c_int
        lib.sf_channel_segment_fwd.argtypes = [dp] + [vp] * 7 + [vp]
        lib.sf_channel_segment_bwd.restype = ctypes.c_int
        lib.sf_channel_segment_bwd.argtypes = [dp] + [vp] * 12 + [vp, sz, vp]
        lib.sf_delta_segment_fwd.restype = ctypes.c_int
        lib.sf_delta_segment_fwd.argtypes = [dp] + [vp] * 8 + [vp]
        lib.sf_delta_segment_bwd.restype = ctypes.c_int
        lib.sf_delta_segment_bwd.argtypes = [dp] + [vp] * 14 + [vp, sz, vp]
        lib.sf_channel_chunked_workspace_bytes.restype = sz
        lib.sf_channel_chunked_workspace_bytes.argtypes = [dp, ctypes.c_int]
        lib.sf_channel_chunked_fwd.restype = ctypes.c_int
        lib.sf_channel_chunked_fwd.argtypes = [dp] + [vp] * 7 + [vp, sz, vp]
        lib.sf_channel_chunked_bwd.restype = ctypes.c_int
        lib.sf_channel_chunked_bwd.argtypes = [dp] + [vp] * 12 + [vp, sz, vp]
        lib.sf_delta_chunked_workspace_bytes.restype = sz
        lib.sf_delta_chunked_workspace_bytes.argtypes = [dp, ctypes.c_int]
        lib.sf_delta_chunked_fwd.restype = ctypes.c_int
        lib.sf_delta_chunked_fwd.argtypes = [dp] + [vp] * 8 + [vp, sz, vp]
        lib.sf_delta_chunked_bwd.restype = ctypes.c_int
        lib.sf_delta_chunked_bwd.argtypes = [dp] + [vp] * 14 + [vp, sz, vp]
        lib.sf_conv_segment_fwd.restype = ctypes.c_int
        lib.sf_conv_segment_fwd.argtypes = [i32] * 4 + [vp] * 5 + [vp]
        lib.sf_conv_segment_bwd.restype = ctypes.c_int
        lib.sf_conv_segment_bwd.argtypes = [i32] * 4 + [vp] * 8 + [vp]
        _lib = lib
    return _lib


def status_string(code: int) -> str:
    return load().sf_status_string(int(code)).decode()


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(code: int, where: str):
    if code != 0:
        raise SfError(code, where)


def make_desc(q: torch.Tensor, v: torch.Tensor, g: torch.Tensor, chunk: int, chunks_per_block: int = 0,
              seg_len: Optional[int] = None) -> SegDesc:
    """Descriptor for q [B,T,H,d_k], v [B,T,H,d_v], g [B,T,H] (views along T are fine)."""
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    if q.stride(3) != 1 or v.stride(3) != 1 or q.stride(2) != dk or v.stride(2) != dv or g.stride(2) != 1:
        raise ValueError("heads and features must be densely packed inside a token")
    dt = {torch.bfloat16: SF_BF16, torch.float32: SF_F32}[q.dtype]
    return SegDesc(B, H, dk, dv, T if seg_len is None else seg_len, chunk, dt, chunks_per_block,
                   q.stride(1), v.stride(1), g.stride(1), q.stride(0), v.stride(0), g.stride(0))


def sf_num_blocks(desc: SegDesc) -> int:
    return int(load().sf_num_blocks(ctypes.byref(desc)))


def sf_workspace_bytes(desc: SegDesc, backward: int) -> int:
    return int(load().sf_workspace_bytes(ctypes.byref(desc), backward))


def _workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


def sf_segment_fwd(desc: SegDesc, q, k, v, g, S_in, o, S_out, workspace: torch.Tensor, stream=None):
    _check(load().sf_segment_fwd(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(S_in), _ptr(o), _ptr(S_out),
                                 _ptr(workspace), workspace.numel(), _stream(stream)), "sf_segment_fwd")


SF_STATIC_SCRATCH_BYTES = 16 << 20


def sf_segment_fwd_static(desc: SegDesc, q, k, v, g, S_in, o, S_out, stream=None):
    """sf_segment_fwd without a workspace argument: for callers that cannot allocate device memory
    (graph capture, no-allocation memory pools, plug-ins that only get input/output pointers).  The
    scratch is a fixed array inside the library; shapes needing more than SF_STATIC_SCRATCH_BYTES
    raise SF_ERR_WORKSPACE.  Calls share the array, so calls that overlap on the GPU race."""
    _check(load().sf_segment_fwd_static(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(S_in), _ptr(o), _ptr(S_out),
                                        _stream(stream)), "sf_segment_fwd_static")


def sf_segment_bwd(desc: SegDesc, q, k, v, g, S_in, dO, dS_out, dq, dk, dv, dg, dS_in, fwd_saved, workspace, stream=None):
    _check(load().sf_segment_bwd(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(S_in), _ptr(dO), _ptr(dS_out),
                                 _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dg), _ptr(dS_in), _ptr(fwd_saved), _ptr(workspace),
                                 workspace.numel(), _stream(stream)), "sf_segment_bwd")


def sf_state_scan(desc: SegDesc, chunks_per_block: int, reverse: bool, log_decay, U, S_boundary_in, states, S_boundary_out,
                  stream=None):
    _check(load().sf_state_scan(ctypes.byref(desc), chunks_per_block, int(reverse), _ptr(log_decay), _ptr(U),
                                _ptr(S_boundary_in), _ptr(states), _ptr(S_boundary_out), _stream(stream)), "sf_state_scan")


def _seg_array(seg_lens: Sequence[int]):
    return (ctypes.c_int32 * len(seg_lens))(*[int(s) for s in seg_lens])


def sf_chain_workspace_bytes(desc: SegDesc, seg_lens: Sequence[int], backward: int) -> int:
    return int(load().sf_chain_workspace_bytes(ctypes.byref(desc), _seg_array(seg_lens), len(seg_lens), backward))


def sf_chain_fwd(desc: SegDesc, seg_lens, q, k, v, g, S_init, o, S_bounds, workspace, overlap=True, stream=None):
    _check(load().sf_chain_fwd(ctypes.byref(desc), _seg_array(seg_lens), len(seg_lens), _ptr(q), _ptr(k), _ptr(v), _ptr(g),
                               _ptr(S_init), _ptr(o), _ptr(S_bounds), _ptr(workspace), workspace.numel(), int(overlap),
                               _stream(stream)), "sf_chain_fwd")


def sf_chain_bwd(desc: SegDesc, seg_lens, q, k, v, g, S_bounds, dO, dS_final, dq, dk, dv, dg, dS_init, fwd_workspace,
                 workspace, overlap=True, stream=None):
    _check(load().sf_chain_bwd(ctypes.byref(desc), _seg_array(seg_lens), len(seg_lens), _ptr(q), _ptr(k), _ptr(v), _ptr(g),
                               _ptr(S_bounds), _ptr(dO), _ptr(dS_final), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dg),
                               _ptr(dS_init), _ptr(fwd_workspace), _ptr(workspace), workspace.numel(), int(overlap),
                               _stream(stream)), "sf_chain_bwd")


def sf_chain_graph_create(desc: SegDesc, seg_lens, q, k, v, g, S_init, o, S_bounds, fwd_workspace, dO, dS_final, dq, dk, dv,
                          dg, dS_init, bwd_workspace, overlap=True, stream=None) -> ctypes.c_void_p:
    """Returns the graph handle; `stream` (default: the current stream) must not be the legacy default stream."""
    handle = ctypes.c_void_p()
    _check(load().sf_chain_graph_create(ctypes.byref(desc), _seg_array(seg_lens), len(seg_lens), _ptr(q), _ptr(k), _ptr(v),
                                        _ptr(g), _ptr(S_init), _ptr(o), _ptr(S_bounds), _ptr(fwd_workspace),
                                        fwd_workspace.numel(), _ptr(dO), _ptr(dS_final), _ptr(dq), _ptr(dk), _ptr(dv),
                                        _ptr(dg), _ptr(dS_init), _ptr(bwd_workspace),
                                        0 if bwd_workspace is None else bwd_workspace.numel(), int(overlap),
                                        _stream(stream), ctypes.byref(handle)), "sf_chain_graph_create")
    return handle


def sf_chain_graph_launch(handle, stream=None) -> None:
    _check(load().sf_chain_graph_launch(handle, _stream(stream)), "sf_chain_graph_launch")


def sf_chain_graph_kernels(handle) -> int:
    return int(load().sf_chain_graph_kernels(handle))


def sf_chain_graph_destroy(handle) -> None:
    load().sf_chain_graph_destroy(handle)


def sf_chain_autotune(desc: SegDesc, seg_lens, q, k, v, g, S_init, o, S_bounds, fwd_workspace, dO, dS_final, dq, dk, dv, dg,
                      dS_init, bwd_workspace, candidates, reps=3, overlap=True, stream=None):
    """Returns (best chunks_per_block, [mean ms per candidate, -1 = skipped])."""
    cand = (ctypes.c_int32 * len(candidates))(*[int(c) for c in candidates])
    ms = (ctypes.c_float * len(candidates))()
    best = ctypes.c_int32(-1)
    _check(load().sf_chain_autotune(ctypes.byref(desc), _seg_array(seg_lens), len(seg_lens), _ptr(q), _ptr(k), _ptr(v),
                                    _ptr(g), _ptr(S_init), _ptr(o), _ptr(S_bounds), _ptr(fwd_workspace),
                                    fwd_workspace.numel(), _ptr(dO), _ptr(dS_final), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dg),
                                    _ptr(dS_init), _ptr(bwd_workspace),
                                    0 if bwd_workspace is None else bwd_workspace.numel(), cand, len(candidates), int(reps),
                                    int(overlap), _stream(stream), ctypes.byref(best), ms), "sf_chain_autotune")
    return int(best.value), [float(x) for x in ms]


def sf_chain_autotune_schedule(desc: SegDesc, seg_lens, q, k, v, g, S_init, o, S_bounds, fwd_workspace, dO, dS_final, dq, dk, dv,
                               dg, dS_init, bwd_workspace, reps=5, margin=0.02, stream=None):
    """Searches the built-in set of schedules, installs the choice (sf_set_tuning) and returns
    (chosen Tuning, chosen ms, default ms)."""
    t = Tuning()
    ms, dms = ctypes.c_float(-1.0), ctypes.c_float(-1.0)
    _check(load().sf_chain_autotune_schedule(ctypes.byref(desc), _seg_array(seg_lens), len(seg_lens), _ptr(q), _ptr(k), _ptr(v),
                                             _ptr(g), _ptr(S_init), _ptr(o), _ptr(S_bounds), _ptr(fwd_workspace),
                                             fwd_workspace.numel(), _ptr(dO), _ptr(dS_final), _ptr(dq), _ptr(dk), _ptr(dv),
                                             _ptr(dg), _ptr(dS_init), _ptr(bwd_workspace), bwd_workspace.numel(), int(reps),
                                             float(margin), _stream(stream), ctypes.byref(t), ctypes.byref(ms), ctypes.byref(dms)),
           "sf_chain_autotune_schedule")
    return t, float(ms.value), float(dms.value)


def sf_partition_hybrid(T: int, N: int, w_tok: float, w_soft: float, alpha: float, multiple: int = 128) -> List[int]:
    """Segment lengths of the candidate partition (host only)."""
    out = (ctypes.c_int32 * max(N, 1))()
    _check(load().sf_partition_hybrid(int(T), int(N), float(w_tok), float(w_soft), float(alpha), int(multiple), out),
           "sf_partition_hybrid")
    return [int(v) for v in out[:N]]


def sf_e2e_device_bytes(desc: SegDesc, seg_lens) -> int:
    return int(load().sf_e2e_device_bytes(ctypes.byref(desc), _seg_array(seg_lens), len(seg_lens)))


def sf_chain_fwd_bwd_host(desc: SegDesc, seg_lens, q, k, v, g, S_init, dO, dS_final, o, S_final, dq, dk, dv, dg, dS_init,
                          dev: torch.Tensor, stream=None):
    """All data tensors are HOST tensors (pinned recommended); dev is device scratch."""
    _check(load().sf_chain_fwd_bwd_host(ctypes.byref(desc), _seg_array(seg_lens), len(seg_lens), _ptr(q), _ptr(k), _ptr(v),
                                        _ptr(g), _ptr(S_init), _ptr(dO), _ptr(dS_final), _ptr(o), _ptr(S_final), _ptr(dq),
                                        _ptr(dk), _ptr(dv), _ptr(dg), _ptr(dS_init), _ptr(dev), dev.numel(),
                                        _stream(stream)), "sf_chain_fwd_bwd_host")


def sf_device_status() -> int:
    return int(load().sf_device_status())


def sf_device_status_clear() -> None:
    load().sf_device_status_clear()


class Tuning(ctypes.Structure):
    """sf_tuning_t: schedule of the chaining driver."""
    _fields_ = [("sweep_streams", ctypes.c_int32), ("agg_streams", ctypes.c_int32), ("scan_group_tokens", ctypes.c_int32),
                ("agg_inorder_ctas", ctypes.c_int32), ("agg_ahead", ctypes.c_int32), ("merge_launches", ctypes.c_int32)]


def sf_set_tuning(tuning=None) -> None:
    """tuning: None (defaults), a Tuning, or a dict with some of its fields (the others keep their current value)."""
    lib = load()
    lib.sf_set_tuning.argtypes = [ctypes.c_void_p]
    if tuning is None:
        _check(lib.sf_set_tuning(None), "sf_set_tuning")
        return
    if isinstance(tuning, dict):
        t = sf_get_tuning()
        for k, v in tuning.items():
            setattr(t, k, int(v))
        tuning = t
    _check(lib.sf_set_tuning(ctypes.byref(tuning)), "sf_set_tuning")


def sf_get_tuning() -> Tuning:
    lib = load()
    lib.sf_get_tuning.argtypes = [ctypes.c_void_p]
    lib.sf_get_tuning.restype = None
    t = Tuning()
    lib.sf_get_tuning(ctypes.byref(t))
    return t


def sf_device_check() -> int:
    """Status code for the device status word: 0 ok, 5 a bounded wait ran out, 4 the word could not be read."""
    return int(load().sf_device_check())


def sf_selftest_bounded_wait(limit_cycles: int = 2_000_000, stream=None) -> int:
    """Runs the wait self-test kernel and returns its status code (5 = SF_ERR_TIMEOUT when the mechanism works)."""
    lib = load()
    lib.sf_selftest_bounded_wait.argtypes = [ctypes.c_int64, ctypes.c_void_p]
    return int(lib.sf_selftest_bounded_wait(int(limit_cycles), _stream(stream)))


def sf_launch_count() -> int:
    return int(load().sf_launch_count())


STAGE_NAMES = ["agg_kv", "agg_qdo", "scan", "fwd_out", "dq", "dkdv", "dg"]


def sf_stage_timing(enable: bool) -> None:
    load().sf_stage_timing(int(enable))


def sf_stage_timing_read():
    n = len(STAGE_NAMES)
    ms = (ctypes.c_float * n)()
    cnt = (ctypes.c_int64 * n)()
    load().sf_stage_timing_read(ms, cnt, n)
    return [{"name": STAGE_NAMES[i], "ms": float(ms[i]), "launches": int(cnt[i])} for i in range(n)]


# ---- extension operators: diagonal decay, gated delta rule, short convolution with a carried tail ----

def sf_recurrent_workspace_bytes(desc: SegDesc) -> int:
    return int(load().sf_recurrent_workspace_bytes(ctypes.byref(desc)))


def sf_channel_segment_fwd(desc: SegDesc, q, k, v, g, S_in, o, S_out, stream=None):
    _check(load().sf_channel_segment_fwd(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(S_in), _ptr(o),
                                         _ptr(S_out), _stream(stream)), "sf_channel_segment_fwd")


def sf_channel_segment_bwd(desc: SegDesc, q, k, v, g, S_in, dO, dS_out, dq, dk, dv, dg, dS_in, workspace, stream=None):
    _check(load().sf_channel_segment_bwd(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(S_in), _ptr(dO),
                                         _ptr(dS_out), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dg), _ptr(dS_in), _ptr(workspace),
                                         workspace.numel(), _stream(stream)), "sf_channel_segment_bwd")


def sf_delta_segment_fwd(desc: SegDesc, q, k, v, g, beta, S_in, o, S_out, stream=None):
    _check(load().sf_delta_segment_fwd(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(S_in), _ptr(o),
                                       _ptr(S_out), _stream(stream)), "sf_delta_segment_fwd")


def sf_delta_segment_bwd(desc: SegDesc, q, k, v, g, beta, S_in, dO, dS_out, dq, dk, dv, dg, dbeta, dS_in, workspace, stream=None):
    _check(load().sf_delta_segment_bwd(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(S_in), _ptr(dO),
                                       _ptr(dS_out), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dg), _ptr(dbeta), _ptr(dS_in),
                                       _ptr(workspace), workspace.numel(), _stream(stream)), "sf_delta_segment_bwd")


def sf_channel_chunked_workspace_bytes(desc: SegDesc, backward: int) -> int:
    return int(load().sf_channel_chunked_workspace_bytes(ctypes.byref(desc), backward))


def sf_channel_chunked_fwd(desc: SegDesc, q, k, v, g, S_in, o, S_out, workspace, stream=None):
    _check(load().sf_channel_chunked_fwd(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(S_in), _ptr(o), _ptr(S_out),
                                         _ptr(workspace), workspace.numel(), _stream(stream)), "sf_channel_chunked_fwd")


def sf_channel_chunked_bwd(desc: SegDesc, q, k, v, g, S_in, dO, dS_out, dq, dk, dv, dg, dS_in, workspace, stream=None):
    _check(load().sf_channel_chunked_bwd(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(S_in), _ptr(dO), _ptr(dS_out),
                                         _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dg), _ptr(dS_in), _ptr(workspace), workspace.numel(),
                                         _stream(stream)), "sf_channel_chunked_bwd")


def sf_delta_chunked_workspace_bytes(desc: SegDesc, backward: int) -> int:
    return int(load().sf_delta_chunked_workspace_bytes(ctypes.byref(desc), backward))


def sf_delta_chunked_fwd(desc: SegDesc, q, k, v, g, beta, S_in, o, S_out, workspace, stream=None):
    _check(load().sf_delta_chunked_fwd(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(S_in), _ptr(o),
                                       _ptr(S_out), _ptr(workspace), workspace.numel(), _stream(stream)), "sf_delta_chunked_fwd")


def sf_delta_chunked_bwd(desc: SegDesc, q, k, v, g, beta, S_in, dO, dS_out, dq, dk, dv, dg, dbeta, dS_in, workspace, stream=None):
    _check(load().sf_delta_chunked_bwd(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(S_in), _ptr(dO),
                                       _ptr(dS_out), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dg), _ptr(dbeta), _ptr(dS_in),
                                       _ptr(workspace), workspace.numel(), _stream(stream)), "sf_delta_chunked_bwd")


def sf_conv_segment_fwd(x, w, tail_in, y, tail_out, stream=None):
    """x, y [B, L, C]; w [W, C]; tails [B, W-1, C]; all dense float32."""
    B, L, C = x.shape
    _check(load().sf_conv_segment_fwd(B, L, C, w.shape[0], _ptr(x), _ptr(w), _ptr(tail_in), _ptr(y), _ptr(tail_out),
                                      _stream(stream)), "sf_conv_segment_fwd")


def sf_conv_segment_bwd(x, w, tail_in, dy, dtail_out, dx, dw, dtail_in, stream=None):
    B, L, C = x.shape
    _check(load().sf_conv_segment_bwd(B, L, C, w.shape[0], _ptr(x), _ptr(w), _ptr(tail_in), _ptr(dy), _ptr(dtail_out), _ptr(dx),
                                      _ptr(dw), _ptr(dtail_in), _stream(stream)), "sf_conv_segment_bwd")


# ---- conveniences built only from the calls above (allocation + one call each) --------------------

class ChainRun:
    """Device buffers for one chained forward+backward over a whole sequence."""

    def __init__(self, q, k, v, g, dO, seg_lens: List[int], chunk: int, chunks_per_block: int = 0, save_states: bool = True):
        self.seg_lens = [int(s) for s in seg_lens]
        self.desc = make_desc(q, v, g, chunk, chunks_per_block, seg_len=self.seg_lens[0])
        dev = q.device
        B, T, H, dk = q.shape
        dv = v.shape[-1]
        self.q, self.k, self.v, self.g, self.dO = q, k, v, g, dO
        self.o = torch.empty_like(v)
        self.dq, self.dk, self.dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        self.dg = torch.empty_like(g)
        self.S_bounds = torch.empty(len(self.seg_lens) + 1, B, H, dk, dv, dtype=torch.float32, device=dev)
        self.dS_init = torch.empty(B, H, dk, dv, dtype=torch.float32, device=dev)
        self.save_states = save_states
        self.ws_f = _workspace(sf_chain_workspace_bytes(self.desc, self.seg_lens, 0), dev)
        self.ws_b = _workspace(sf_chain_workspace_bytes(self.desc, self.seg_lens, 1 if save_states else 2), dev)

    def forward(self, S_init=None, overlap=True, stream=None):
        sf_chain_fwd(self.desc, self.seg_lens, self.q, self.k, self.v, self.g, S_init, self.o, self.S_bounds, self.ws_f,
                     overlap, stream)

    def backward(self, dS_final=None, overlap=True, stream=None):
        sf_chain_bwd(self.desc, self.seg_lens, self.q, self.k, self.v, self.g, self.S_bounds, self.dO, dS_final, self.dq,
                     self.dk, self.dv, self.dg, self.dS_init, self.ws_f if self.save_states else None, self.ws_b, overlap,
                     stream)

    def capture(self, S_init=None, dS_final=None, overlap=True, stream=None):
        """Records forward + backward as one CUDA graph (needs saved states); S_init / dS_final must stay alive."""
        if not self.save_states:
            raise ValueError("graph capture needs the forward workspace")
        self.release()
        self._graph_keep = (S_init, dS_final)
        self.graph = sf_chain_graph_create(self.desc, self.seg_lens, self.q, self.k, self.v, self.g, S_init, self.o,
                                           self.S_bounds, self.ws_f, self.dO, dS_final, self.dq, self.dk, self.dv, self.dg,
                                           self.dS_init, self.ws_b, overlap, stream)
        return sf_chain_graph_kernels(self.graph)

    def replay(self, stream=None):
        sf_chain_graph_launch(self.graph, stream)

    def release(self):
        if getattr(self, "graph", None) is not None:
            sf_chain_graph_destroy(self.graph)
            self.graph = None

    def __del__(self):
        try:
            self.release()
        except Exception:
            pass

    def autotune_schedule(self, S_init=None, dS_final=None, reps=5, margin=0.02, stream=None):
        """Profile-guided schedule of the chain driver for these buffers; the choice stays installed process-wide."""
        self.release()
        return sf_chain_autotune_schedule(self.desc, self.seg_lens, self.q, self.k, self.v, self.g, S_init, self.o, self.S_bounds,
                                          self.ws_f, self.dO, dS_final, self.dq, self.dk, self.dv, self.dg, self.dS_init,
                                          self.ws_b, reps, margin, stream)

    def autotune(self, S_init=None, dS_final=None, candidates=(0, 8, 10, 11, 13, 16, 19, 22, 26, 29, 32), reps=3, overlap=True, stream=None):
        """Times the chain for every candidate block length, keeps the fastest in the descriptor and returns
        (best, [ms per candidate]).  Workspaces are re-allocated for the candidate with the most blocks."""
        if not self.save_states:
            raise ValueError("tuning runs the backward from saved states")
        self.release()
        dev = self.q.device
        need_f = need_b = 0
        keep = self.desc.chunks_per_block
        for c in candidates:
            self.desc.chunks_per_block = int(c)
            need_f = max(need_f, sf_chain_workspace_bytes(self.desc, self.seg_lens, 0))
            need_b = max(need_b, sf_chain_workspace_bytes(self.desc, self.seg_lens, 1))
        self.desc.chunks_per_block = keep
        self.ws_f, self.ws_b = _workspace(need_f, dev), _workspace(need_b, dev)
        best, ms = sf_chain_autotune(self.desc, self.seg_lens, self.q, self.k, self.v, self.g, S_init, self.o, self.S_bounds,
                                     self.ws_f, self.dO, dS_final, self.dq, self.dk, self.dv, self.dg, self.dS_init,
                                     self.ws_b, candidates, reps, overlap, stream)
        self.desc.chunks_per_block = best
        return best, ms
