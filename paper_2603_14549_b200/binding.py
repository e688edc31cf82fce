"""ctypes binding of libasap.so: same names as the C entry points, argument marshalling only.

Every step of the prune path runs in the CUDA library.  PyTorch is used here for device
memory (the tensors whose data pointers are handed to the library) and for the current
stream.  There is no CPU fallback: if the library is missing or was not built, loading
raises.
"""
from __future__ import annotations

import ctypes as C
import dataclasses
import math
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libasap.so")

ASAP_OK = 0
STATUS_NAMES = {0: "ASAP_OK", -1: "ASAP_ERR_INVALID", -2: "ASAP_ERR_ALIGN", -3: "ASAP_ERR_WORKSPACE",
                -4: "ASAP_ERR_CUDA", -5: "ASAP_ERR_UNSUPPORTED", -6: "ASAP_ERR_DEVICE"}

EXPORTS = ("asap_init", "asap_score", "asap_select", "asap_merge", "asap_prune_step", "asap_check",
           "asap_last_error", "asap_launch_count", "asap_free", "asap_profile", "asap_profile_read", "asap_debug_wait_limit", "asap_select_static", "asap_compact_kv",
           "asap_consolidate", "asap_consolidate_scratch_bytes", "asap_attention", "asap_attention_scratch_bytes")


class AsapError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {text}")
        self.status = status


class CInputs(C.Structure):
    _fields_ = [("B", C.c_int32), ("H", C.c_int32), ("head_dim", C.c_int32), ("D", C.c_int32),
                ("total_tokens", C.c_int32), ("min_vis", C.c_int32), ("max_vis", C.c_int32),
                ("max_seq", C.c_int32), ("max_rank", C.c_int32),
                ("cu_seqlens", C.c_void_p), ("vis_start", C.c_void_p), ("vis_len", C.c_void_p),
                ("text_start", C.c_void_p), ("text_len", C.c_void_p), ("rank_start", C.c_void_p),
                ("rank_len", C.c_void_p), ("q", C.c_void_p), ("k", C.c_void_p), ("hidden", C.c_void_p),
                ("pos_ids", C.c_void_p)]


class CParams(C.Structure):
    _fields_ = [("keep_k", C.c_int32), ("lambda_max", C.c_float), ("eps", C.c_float),
                ("sim_threshold", C.c_float), ("mask_enable", C.c_int32), ("merge_enable", C.c_int32),
                ("per_head_mask", C.c_int32)]


class CKernelTime(C.Structure):
    _fields_ = [("name", C.c_char * 32), ("launches", C.c_uint64), ("total_ms", C.c_double)]


class COutputs(C.Structure):
    _fields_ = [("mass", C.c_void_p), ("salience", C.c_void_p), ("mask_log", C.c_void_p),
                ("rank_score", C.c_void_p), ("keep_idx", C.c_void_p), ("drop_idx", C.c_void_p),
                ("assign", C.c_void_p), ("best_sim", C.c_void_p), ("out_hidden", C.c_void_p),
                ("out_pos", C.c_void_p), ("src_row", C.c_void_p), ("out_cu_seqlens", C.c_void_p),
                ("out_rows_capacity", C.c_int32), ("mask_log_heads", C.c_void_p)]


_lib = None


def load_library() -> C.CDLL:
    """Loads libasap.so; raises if it has not been built (python -m paper_2603_14549_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} is missing: build it with `python paper_2603_14549_b200/build.py` "
            "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    lib.asap_init.restype = C.c_int
    lib.asap_init.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_size_t, C.c_int, C.c_int, C.c_int, C.c_size_t]
    for name in ("asap_score", "asap_prune_step"):
        fn = getattr(lib, name)
        fn.restype = C.c_int
        fn.argtypes = [C.c_void_p, C.POINTER(CInputs), C.POINTER(CParams), C.POINTER(COutputs), C.c_void_p]
    lib.asap_select.restype = C.c_int
    lib.asap_select.argtypes = [C.c_void_p, C.POINTER(CInputs), C.POINTER(CParams), C.c_void_p,
                                C.POINTER(COutputs), C.c_void_p]
    lib.asap_merge.restype = C.c_int
    lib.asap_merge.argtypes = [C.c_void_p, C.POINTER(CInputs), C.POINTER(CParams), C.c_void_p, C.c_void_p,
                               C.c_void_p, C.POINTER(COutputs), C.c_void_p]
    lib.asap_select_static.restype = C.c_int
    lib.asap_select_static.argtypes = [C.POINTER(CInputs), C.POINTER(CParams), C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.c_void_p, C.c_void_p]
    lib.asap_compact_kv.restype = C.c_int
    lib.asap_compact_kv.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_size_t, C.c_int32,
                                    C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.c_void_p]
    lib.asap_consolidate_scratch_bytes.restype = C.c_size_t
    lib.asap_consolidate_scratch_bytes.argtypes = [C.c_int32, C.c_int32]
    lib.asap_consolidate.restype = C.c_int
    lib.asap_consolidate.argtypes = [C.c_void_p, C.POINTER(CInputs), C.POINTER(CParams), C.c_void_p, C.c_void_p,
                                     C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.POINTER(COutputs),
                                     C.c_void_p, C.c_void_p]
    lib.asap_attention_scratch_bytes.restype = C.c_size_t
    lib.asap_attention_scratch_bytes.argtypes = [C.c_int32, C.c_int32]
    lib.asap_attention.restype = C.c_int
    lib.asap_attention.argtypes = [C.c_void_p, C.POINTER(CInputs), C.POINTER(CParams), C.c_void_p, C.c_void_p,
                                   C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
    lib.asap_check.restype = C.c_int
    lib.asap_check.argtypes = [C.c_void_p, C.c_void_p]
    lib.asap_last_error.restype = C.c_char_p
    lib.asap_last_error.argtypes = [C.c_void_p]
    lib.asap_launch_count.restype = C.c_uint64
    lib.asap_launch_count.argtypes = [C.c_void_p]
    lib.asap_profile.restype = C.c_int
    lib.asap_profile.argtypes = [C.c_void_p, C.c_int]
    lib.asap_debug_wait_limit.restype = C.c_int
    lib.asap_debug_wait_limit.argtypes = [C.c_void_p, C.c_longlong]
    lib.asap_profile_read.restype = C.c_int
    lib.asap_profile_read.argtypes = [C.c_void_p, C.POINTER(CKernelTime), C.c_int]
    lib.asap_free.restype = None
    lib.asap_free.argtypes = [C.c_void_p]
    _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


@dataclasses.dataclass
class Inputs:
    """Device tensors plus the host-known sizes of one packed batch."""
    B: int
    H: int
    head_dim: int
    D: int
    total_tokens: int
    min_vis: int
    max_vis: int
    max_seq: int
    max_rank: int
    cu_seqlens: torch.Tensor
    vis_start: torch.Tensor
    vis_len: torch.Tensor
    text_start: torch.Tensor
    text_len: torch.Tensor
    q: Optional[torch.Tensor]
    k: Optional[torch.Tensor]
    hidden: Optional[torch.Tensor]
    pos_ids: Optional[torch.Tensor]
    rank_start: Optional[torch.Tensor] = None
    rank_len: Optional[torch.Tensor] = None

    def c_struct(self) -> CInputs:
        return CInputs(self.B, self.H, self.head_dim, self.D, self.total_tokens, self.min_vis, self.max_vis,
                       self.max_seq, self.max_rank, _ptr(self.cu_seqlens), _ptr(self.vis_start),
                       _ptr(self.vis_len), _ptr(self.text_start), _ptr(self.text_len), _ptr(self.rank_start),
                       _ptr(self.rank_len), _ptr(self.q), _ptr(self.k), _ptr(self.hidden), _ptr(self.pos_ids))


def make_inputs(batch, device, rank_start=None, rank_len=None) -> Inputs:
    """Moves a workloads.Batch to `device` and derives the host-known bounds."""
    dev = lambda t: t.to(device, non_blocking=False).contiguous()
    seq = (batch.cu_seqlens[1:] - batch.cu_seqlens[:-1])
    rl = batch.text_len if rank_len is None else torch.as_tensor(rank_len, dtype=torch.int32)
    rs = None if rank_start is None else torch.as_tensor(rank_start, dtype=torch.int32)
    return Inputs(B=batch.B, H=batch.H, head_dim=batch.head_dim, D=batch.D, total_tokens=batch.total,
                  min_vis=int(batch.vis_len.min()), max_vis=int(batch.vis_len.max()), max_seq=int(seq.max()),
                  max_rank=int(rl.max()), cu_seqlens=dev(batch.cu_seqlens), vis_start=dev(batch.vis_start),
                  vis_len=dev(batch.vis_len), text_start=dev(batch.text_start), text_len=dev(batch.text_len),
                  q=dev(batch.q), k=dev(batch.k), hidden=dev(batch.hidden), pos_ids=dev(batch.pos_ids),
                  rank_start=None if rs is None else dev(rs),
                  rank_len=None if rank_len is None else dev(rl))


@dataclasses.dataclass
class Params:
    keep_k: int
    lambda_max: float = 1.0
    eps: float = 1e-6
    sim_threshold: float = -math.inf
    mask_enable: bool = True
    merge_enable: bool = True
    per_head_mask: bool = False

    def c_struct(self) -> CParams:
        return CParams(self.keep_k, self.lambda_max, self.eps, self.sim_threshold, int(self.mask_enable),
                       int(self.merge_enable), int(self.per_head_mask))


@dataclasses.dataclass
class Outputs:
    mass: torch.Tensor
    salience: torch.Tensor
    mask_log: torch.Tensor
    rank_score: torch.Tensor
    keep_idx: torch.Tensor
    drop_idx: torch.Tensor
    assign: torch.Tensor
    best_sim: Optional[torch.Tensor]
    out_hidden: torch.Tensor
    out_pos: torch.Tensor
    src_row: torch.Tensor
    out_cu_seqlens: torch.Tensor
    mask_log_heads: Optional[torch.Tensor] = None

    def c_struct(self) -> COutputs:
        return COutputs(_ptr(self.mass), _ptr(self.salience), _ptr(self.mask_log), _ptr(self.rank_score),
                        _ptr(self.keep_idx), _ptr(self.drop_idx), _ptr(self.assign), _ptr(self.best_sim),
                        _ptr(self.out_hidden), _ptr(self.out_pos), _ptr(self.src_row),
                        _ptr(self.out_cu_seqlens), int(self.out_hidden.shape[0]), _ptr(self.mask_log_heads))


def alloc_outputs(inp: Inputs, keep_k: int, best_sim: bool = True, fill: bool = False,
                  per_head: bool = False) -> Outputs:
    """Caller-owned output tensors with the capacities the header states."""
    dev = inp.cu_seqlens.device
    B, mv = inp.B, inp.max_vis
    nd = max(mv - keep_k, 0)
    rows = inp.total_tokens - B * (inp.min_vis - keep_k)
    f32 = lambda *s: (torch.full(s, float("nan"), dtype=torch.float32, device=dev) if fill
                      else torch.empty(s, dtype=torch.float32, device=dev))
    i32 = lambda *s: (torch.full(s, -7, dtype=torch.int32, device=dev) if fill
                      else torch.empty(s, dtype=torch.int32, device=dev))
    return Outputs(mass=f32(B, mv), salience=f32(B, mv), mask_log=f32(B, mv), rank_score=f32(B, mv),
                   keep_idx=i32(B, keep_k), drop_idx=i32(B, nd), assign=i32(B, nd),
                   best_sim=f32(B, nd) if best_sim else None,
                   out_hidden=torch.zeros(rows, inp.D, dtype=torch.bfloat16, device=dev) if fill
                   else torch.empty(rows, inp.D, dtype=torch.bfloat16, device=dev),
                   out_pos=i32(rows), src_row=i32(rows), out_cu_seqlens=i32(B + 1),
                   mask_log_heads=f32(B, inp.H, mv) if per_head else None)


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _raise(ctx, status: int):
    if status != ASAP_OK:
        text = load_library().asap_last_error(ctx)
        raise AsapError(status, text.decode() if text else "")


# ------------------------------------------------------------------------------------ entry points
def asap_init(device: int, max_total_tokens: int, max_B: int, max_H: int, max_D: int,
              max_keep_rows: int = 0) -> C.c_void_p:
    lib = load_library()
    ctx = C.c_void_p()
    st = lib.asap_init(C.byref(ctx), int(device), int(max_total_tokens), int(max_B), int(max_H), int(max_D),
                       int(max_keep_rows))
    _raise(None, st)
    return ctx


def asap_score(ctx, inp: Inputs, params: Params, out: Outputs, stream=None) -> None:
    ci, cp, co = inp.c_struct(), params.c_struct(), out.c_struct()
    _raise(ctx, load_library().asap_score(ctx, C.byref(ci), C.byref(cp), C.byref(co), _stream(stream)))


def asap_select(ctx, inp: Inputs, params: Params, rank_score: torch.Tensor, out: Outputs, stream=None) -> None:
    ci, cp, co = inp.c_struct(), params.c_struct(), out.c_struct()
    _raise(ctx, load_library().asap_select(ctx, C.byref(ci), C.byref(cp), _ptr(rank_score), C.byref(co),
                                           _stream(stream)))


def asap_select_static(inp: Inputs, params: Params, rank_score: torch.Tensor, keep_idx: torch.Tensor,
                       drop_idx: Optional[torch.Tensor], device_status: Optional[torch.Tensor] = None,
                       stream=None) -> None:
    """Top-k selection without a context: the library's fixed device array is the scratch, so
    nothing is allocated.  Works on the current CUDA device; B <= 64, B * max_vis <= 262144."""
    ci, cp = inp.c_struct(), params.c_struct()
    _raise(None, load_library().asap_select_static(C.byref(ci), C.byref(cp), _ptr(rank_score), _ptr(keep_idx),
                                                   _ptr(drop_idx), _ptr(device_status), _stream(stream)))


def asap_merge(ctx, inp: Inputs, params: Params, salience: torch.Tensor, keep_idx: torch.Tensor,
               drop_idx: torch.Tensor, out: Outputs, stream=None) -> None:
    ci, cp, co = inp.c_struct(), params.c_struct(), out.c_struct()
    _raise(ctx, load_library().asap_merge(ctx, C.byref(ci), C.byref(cp), _ptr(salience), _ptr(keep_idx),
                                          _ptr(drop_idx), C.byref(co), _stream(stream)))


def asap_attention_scratch_bytes(total_tokens: int, D: int) -> int:
    return int(load_library().asap_attention_scratch_bytes(int(total_tokens), int(D)))


def asap_attention(ctx, inp: Inputs, params: Params, mask_log: Optional[torch.Tensor], v: torch.Tensor,
                   scratch: torch.Tensor, out: torch.Tensor, stream=None) -> None:
    """out[i, h, :] = sum_j Softmax_j(q_i.k_j / sqrt(d) + M_ij) v_j; `v`, `out`: bf16 [total_tokens, H, head_dim]."""
    ci, cp = inp.c_struct(), params.c_struct()
    _raise(ctx, load_library().asap_attention(ctx, C.byref(ci), C.byref(cp), _ptr(mask_log), _ptr(v), _ptr(scratch),
                                              int(scratch.numel() * scratch.element_size()), _ptr(out), _stream(stream)))


def asap_consolidate_scratch_bytes(B: int, keep_k: int) -> int:
    return int(load_library().asap_consolidate_scratch_bytes(int(B), int(keep_k)))


def asap_consolidate(ctx, inp: Inputs, params: Params, mass: torch.Tensor, salience: torch.Tensor,
                     keep_idx: torch.Tensor, drop_idx: torch.Tensor, scratch: torch.Tensor, out: Outputs,
                     n_absorbed: Optional[torch.Tensor] = None, stream=None) -> None:
    """`scratch`: a contiguous device tensor of at least asap_consolidate_scratch_bytes(B, keep_k) bytes."""
    ci, cp, co = inp.c_struct(), params.c_struct(), out.c_struct()
    _raise(ctx, load_library().asap_consolidate(
        ctx, C.byref(ci), C.byref(cp), _ptr(mass), _ptr(salience), _ptr(keep_idx), _ptr(drop_idx), _ptr(scratch),
        int(scratch.numel() * scratch.element_size()), C.byref(co), _ptr(n_absorbed), _stream(stream)))


def asap_prune_step(ctx, inp: Inputs, params: Params, out: Outputs, stream=None) -> None:
    ci, cp, co = inp.c_struct(), params.c_struct(), out.c_struct()
    _raise(ctx, load_library().asap_prune_step(ctx, C.byref(ci), C.byref(cp), C.byref(co), _stream(stream)))


def asap_compact_kv(ctx, src_row: torch.Tensor, n_rows: torch.Tensor, src, dst, stream=None) -> None:
    """dst[t][r] = src[t][src_row[r]] for r < n_rows[0]: `src` / `dst` are equally long lists of 2-D device
    tensors (rows x anything, contiguous); `n_rows` is a one-element int32 device tensor (or a view
    such as out_cu_seqlens[B:])."""
    assert len(src) == len(dst) and len(src) > 0
    row_bytes = src[0][0].numel() * src[0].element_size()
    ps = (C.c_void_p * len(src))(*[t.data_ptr() for t in src])
    pd = (C.c_void_p * len(dst))(*[t.data_ptr() for t in dst])
    _raise(ctx, load_library().asap_compact_kv(ctx, _ptr(src_row), _ptr(n_rows), int(min(dst[0].shape[0], src_row.numel())),
                                               int(src[0].shape[0]), int(row_bytes), len(src), ps, pd, _stream(stream)))


def asap_check(ctx, stream=None) -> None:
    _raise(ctx, load_library().asap_check(ctx, _stream(stream)))


def asap_launch_count(ctx) -> int:
    return int(load_library().asap_launch_count(ctx))


def asap_last_error(ctx) -> str:
    text = load_library().asap_last_error(ctx)
    return text.decode() if text else ""


def asap_debug_wait_limit(ctx, cycles: int) -> None:
    _raise(ctx, load_library().asap_debug_wait_limit(ctx, int(cycles)))


def asap_profile(ctx, enable: bool) -> None:
    _raise(ctx, load_library().asap_profile(ctx, int(bool(enable))))


def asap_profile_read(ctx) -> dict:
    """{kernel name: (launches, total_ms)} accumulated since profiling was enabled."""
    buf = (CKernelTime * 32)()
    n = load_library().asap_profile_read(ctx, buf, 32)
    return {buf[i].name.decode(): (int(buf[i].launches), float(buf[i].total_ms)) for i in range(min(n, 32))}


def asap_free(ctx) -> None:
    load_library().asap_free(ctx)
