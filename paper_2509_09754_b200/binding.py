"""ctypes binding of liblava.so: argument marshalling only."""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

LAVA_F32, LAVA_BF16 = 0, 1
LAVA_POOL_NONE, LAVA_POOL_MAX, LAVA_POOL_AVG = 0, 1, 2
LAVA_BUDGET_DYNAMIC, LAVA_BUDGET_UNIFORM, LAVA_BUDGET_PYRAMID = 0, 1, 2
LAVA_FLAG_PER_HEAD_TOPK, LAVA_FLAG_UNIT_VALUE_NORM, LAVA_FLAG_TOKEN_VALUE_NORM = 1, 2, 4

_STATUS_NAMES = {0: "LAVA_OK", 1: "LAVA_ERR_INVALID_ARG", 2: "LAVA_ERR_UNSUPPORTED",
                 3: "LAVA_ERR_WORKSPACE", 4: "LAVA_ERR_CUDA", 5: "LAVA_ERR_TIMEOUT"}


class LavaError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("%s: %s" % (_STATUS_NAMES.get(status, str(status)), message))
        self.status = status


class _CDesc(ctypes.Structure):
    _fields_ = [
        ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("window", ctypes.c_int32),
        ("pool_kind", ctypes.c_int32), ("pool_kernel", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("batch", ctypes.c_int32),
        ("max_seqlen", ctypes.c_int32), ("flags", ctypes.c_int32),
        ("cu_seqlens", ctypes.c_void_p), ("total_tokens", ctypes.c_int64),
        ("k_stride_head", ctypes.c_int64), ("k_stride_tok", ctypes.c_int64),
        ("v_stride_head", ctypes.c_int64), ("v_stride_tok", ctypes.c_int64),
        ("sm_scale", ctypes.c_float), ("c_hat", ctypes.c_float),
    ]


class _CCascadeView(ctypes.Structure):
    _fields_ = [
        ("layers_done", ctypes.c_int32), ("k_out", ctypes.c_void_p), ("v_out", ctypes.c_void_p),
        ("kept_pos", ctypes.c_void_p), ("kept_scores", ctypes.c_void_p),
        ("head_offsets", ctypes.c_void_p), ("layer_budget", ctypes.c_void_p),
        ("layer_row_offset", ctypes.c_void_p), ("entropy", ctypes.c_void_p),
    ]


_LIB = None


def library_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "lib", "liblava.so")


def load_library():
    """Load liblava.so; raises if it has not been built (there is no fallback path)."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise RuntimeError(
            "liblava.so is missing (%s): build it with `python -m paper_2509_09754_b200.build`; "
            "this package has no CPU or PyTorch fallback" % path)
    lib = ctypes.CDLL(path)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    dp = ctypes.POINTER(_CDesc)
    lib.lava_version.restype = i32
    lib.lava_last_error.restype = ctypes.c_char_p
    lib.lava_workspace_bytes.restype = sz
    lib.lava_workspace_bytes.argtypes = [dp, i32]
    lib.lava_poll_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.lava_wo_norm.argtypes = [vp, i32, i64, i64, vp, vp]
    lib.lava_score_layer.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.lava_score_layer_static.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.lava_score_layer_static.restype = i32
    lib.lava_score_layers.argtypes = [dp, i32, vp, vp, vp, i64, i64, i64, vp, vp, vp, vp, vp, sz, vp]
    lib.lava_layer_budgets.argtypes = [i32, i32, vp, vp, vp, vp, i32, vp, vp, vp, vp]
    lib.lava_select_topk.argtypes = [dp, vp, vp, vp, vp, vp, sz, vp]
    lib.lava_select_topk_layers.argtypes = [dp, i32, vp, vp, vp, vp, vp, sz, vp]
    lib.lava_compact_kv.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.lava_compact_kv_layers.argtypes = [dp, i32, vp, vp, i64, i64, vp, vp, vp, vp, vp, vp]
    lib.lava_host_arena_bytes.restype = sz
    lib.lava_host_arena_bytes.argtypes = [dp, i32, i64]
    lib.lava_evict_model_host.argtypes = [dp, i32, vp, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp]
    lib.lava_evict_model_host.restype = i32
    lib.lava_launch_count.restype = i64
    lib.lava_launch_count.argtypes = []
    lib.lava_score_path.restype = i32
    lib.lava_score_path.argtypes = [dp]
    lib.lava_set_option.restype = i32
    lib.lava_set_option.argtypes = [ctypes.c_char_p, i64]
    lib.lava_get_option.restype = i64
    lib.lava_get_option.argtypes = [ctypes.c_char_p]
    lib.lava_select_shard_bytes.restype = sz
    lib.lava_select_shard_bytes.argtypes = [dp, i32]
    szp = ctypes.POINTER(sz)
    lib.lava_select_shard_layout.argtypes = [dp, i32, szp, szp, szp, szp]
    lib.lava_select_shard_begin.argtypes = [dp, i32, i32, vp, vp, sz, vp]
    lib.lava_select_shard_hist.argtypes = [dp, i32, vp, i32, vp, sz, vp]
    lib.lava_select_shard_step.argtypes = [dp, i32, i32, vp, sz, vp]
    lib.lava_select_shard_count.argtypes = [dp, i32, vp, vp, sz, vp]
    lib.lava_select_shard_emit.argtypes = [dp, i32, vp, vp, vp, vp, vp, vp, sz, vp]
    for name in ("lava_select_shard_layout", "lava_select_shard_begin", "lava_select_shard_hist",
                 "lava_select_shard_step", "lava_select_shard_count", "lava_select_shard_emit"):
        getattr(lib, name).restype = i32
    lib.lava_decode_workspace_bytes.restype = sz
    lib.lava_decode_workspace_bytes.argtypes = [dp, i32]
    lib.lava_decode_attention_layers.restype = i32
    lib.lava_decode_attention_layers.argtypes = [dp, i32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.lava_decode_attention.restype = i32
    lib.lava_decode_attention.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.lava_loss_workspace_bytes.restype = sz
    lib.lava_loss_workspace_bytes.argtypes = [dp, i64]
    lib.lava_layer_output_loss.restype = i32
    lib.lava_layer_output_loss.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, i32, i64, vp, vp, vp, sz, vp]
    lib.lava_cascade_state_bytes.restype = sz
    lib.lava_cascade_state_bytes.argtypes = [dp, i32, i64]
    lib.lava_cascade_create.argtypes = [dp, i32, i64, i32, vp, sz, ctypes.POINTER(vp)]
    lib.lava_cascade_destroy.restype = None
    lib.lava_cascade_destroy.argtypes = [vp]
    lib.lava_cascade_begin.argtypes = [vp, vp, vp, vp]
    lib.lava_cascade_step.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp]
    lib.lava_cascade_get.argtypes = [vp, ctypes.POINTER(_CCascadeView)]
    for name in ("lava_cascade_create", "lava_cascade_begin", "lava_cascade_step", "lava_cascade_get"):
        getattr(lib, name).restype = i32
    for name in ("lava_poll_status", "lava_wo_norm", "lava_score_layer", "lava_score_layers",
                 "lava_layer_budgets", "lava_select_topk", "lava_select_topk_layers",
                 "lava_compact_kv", "lava_compact_kv_layers"):
        getattr(lib, name).restype = i32
    _LIB = lib
    return lib


def _check(status: int):
    if status != 0:
        raise LavaError(status, load_library().lava_last_error().decode("utf-8", "replace"))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return LAVA_F32
    if t.dtype == torch.bfloat16:
        return LAVA_BF16
    raise LavaError(2, "unsupported tensor dtype %s" % t.dtype)


@dataclass
class LayerDesc:
    """Host-side mirror of lava_layer_desc.  K/V layout: [H_kv, total_tokens, d] views with
    arbitrary head/token strides (last dim contiguous)."""
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    window: int
    pool_kind: int = LAVA_POOL_MAX
    pool_kernel: int = 7
    dtype: int = LAVA_BF16
    batch: int = 1
    max_seqlen: int = 0
    cu_seqlens: Optional[torch.Tensor] = None     # device int32 [batch + 1]
    total_tokens: int = 0
    k_stride_head: int = 0
    k_stride_tok: int = 0
    v_stride_head: int = 0
    v_stride_tok: int = 0
    sm_scale: float = 0.0
    c_hat: float = 0.0
    flags: int = 0

    @staticmethod
    def for_tensors(q_win: torch.Tensor, k: torch.Tensor, v: Optional[torch.Tensor], window: int,
                    pool_kind: int = LAVA_POOL_MAX, pool_kernel: int = 7,
                    cu_seqlens: Optional[torch.Tensor] = None, max_seqlen: int = 0,
                    sm_scale: float = 0.0, c_hat: float = 0.0, flags: int = 0) -> "LayerDesc":
        """q_win [batch, H_q, w, d]; k, v [H_kv, total_tokens, d] (one layer's views)."""
        batch, hq, w, d = q_win.shape
        hkv, total, _ = k.shape
        vv = v if v is not None else k
        return LayerDesc(
            n_q_heads=hq, n_kv_heads=hkv, head_dim=d, window=window, pool_kind=pool_kind,
            pool_kernel=pool_kernel, dtype=_dtype_code(k), batch=batch, max_seqlen=max_seqlen,
            cu_seqlens=cu_seqlens, total_tokens=total, k_stride_head=k.stride(0),
            k_stride_tok=k.stride(1), v_stride_head=vv.stride(0), v_stride_tok=vv.stride(1),
            sm_scale=sm_scale, c_hat=c_hat, flags=flags)

    @property
    def total_scores(self) -> int:
        return self.n_kv_heads * (self.total_tokens - self.batch * self.window)

    def to_c(self) -> _CDesc:
        return _CDesc(self.n_q_heads, self.n_kv_heads, self.head_dim, self.window, self.pool_kind,
                      self.pool_kernel, self.dtype, self.batch, self.max_seqlen, self.flags,
                      None if self.cu_seqlens is None else self.cu_seqlens.data_ptr(),
                      self.total_tokens, self.k_stride_head, self.k_stride_tok,
                      self.v_stride_head, self.v_stride_tok, self.sm_scale, self.c_hat)


# ----------------------------------------------------------------------------- plumbing
def lava_version() -> int:
    return int(load_library().lava_version())


def lava_last_error() -> str:
    return load_library().lava_last_error().decode("utf-8", "replace")


def lava_workspace_bytes(desc: LayerDesc, n_layers: int = 1) -> int:
    c = desc.to_c()
    n = int(load_library().lava_workspace_bytes(ctypes.byref(c), n_layers))
    if n == 0:
        raise LavaError(1, lava_last_error())
    return n


def lava_poll_status(workspace: torch.Tensor, stream=None) -> int:
    word = ctypes.c_uint32(0)
    _check(load_library().lava_poll_status(_ptr(workspace), _stream(stream), ctypes.byref(word)))
    return int(word.value)


def lava_wo_norm(w_o: torch.Tensor, c_hat_out: torch.Tensor, stream=None) -> None:
    rows, cols = w_o.shape
    _check(load_library().lava_wo_norm(_ptr(w_o), _dtype_code(w_o), rows, cols, _ptr(c_hat_out),
                                       _stream(stream)))


# ----------------------------------------------------------------------------- the four steps
def lava_score_layer(desc: LayerDesc, q_win, k, v, vbar_in, scores, vbar_out, entropy, workspace,
                     stream=None) -> None:
    c = desc.to_c()
    _check(load_library().lava_score_layer(
        ctypes.byref(c), _ptr(q_win), _ptr(k), _ptr(v), _ptr(vbar_in), _ptr(scores),
        _ptr(vbar_out), _ptr(entropy), _ptr(workspace), workspace.numel() * workspace.element_size(),
        _stream(stream)))


def lava_score_layer_static(desc: LayerDesc, q_win, k, v, vbar_in, scores, vbar_out, entropy,
                            device_status_out=None, stream=None) -> None:
    """lava_score_layer without a workspace argument, for callers that cannot allocate device
    memory (the scratch is an 8 MiB array inside the library; larger layers are rejected).
    Calls on one device must not overlap on the GPU: keep them on one stream."""
    c = desc.to_c()
    _check(load_library().lava_score_layer_static(
        ctypes.byref(c), _ptr(q_win), _ptr(k), _ptr(v), _ptr(vbar_in), _ptr(scores),
        _ptr(vbar_out), _ptr(entropy), _ptr(device_status_out), _stream(stream)))


def lava_score_layers(desc: LayerDesc, n_layers, q_win, k, v, q_layer_stride, k_layer_stride,
                      v_layer_stride, vbar_in, scores, vbar_out, entropy, workspace,
                      stream=None) -> None:
    c = desc.to_c()
    _check(load_library().lava_score_layers(
        ctypes.byref(c), n_layers, _ptr(q_win), _ptr(k), _ptr(v), q_layer_stride, k_layer_stride,
        v_layer_stride, _ptr(vbar_in), _ptr(scores), _ptr(vbar_out), _ptr(entropy),
        _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))


def lava_layer_budgets(n_layers, batch, entropy, total_budget, floor_per_layer, cap_per_layer,
                       mode, layer_budget, layer_row_offset, status_word=None, stream=None) -> None:
    _check(load_library().lava_layer_budgets(
        n_layers, batch, _ptr(entropy), _ptr(total_budget), _ptr(floor_per_layer),
        _ptr(cap_per_layer), mode, _ptr(layer_budget), _ptr(layer_row_offset), _ptr(status_word),
        _stream(stream)))


def _ws_args(workspace):
    if workspace is None:
        return None, 0
    return _ptr(workspace), workspace.numel() * workspace.element_size()


def lava_select_topk(desc: LayerDesc, scores, layer_budget, keep_idx, head_offsets,
                     workspace=None, stream=None) -> None:
    c = desc.to_c()
    wp, wb = _ws_args(workspace)
    _check(load_library().lava_select_topk(ctypes.byref(c), _ptr(scores), _ptr(layer_budget),
                                           _ptr(keep_idx), _ptr(head_offsets), wp, wb,
                                           _stream(stream)))


def lava_select_topk_layers(desc: LayerDesc, n_layers, scores, layer_budget, keep_idx,
                            head_offsets, workspace=None, stream=None) -> None:
    c = desc.to_c()
    wp, wb = _ws_args(workspace)
    _check(load_library().lava_select_topk_layers(
        ctypes.byref(c), n_layers, _ptr(scores), _ptr(layer_budget), _ptr(keep_idx),
        _ptr(head_offsets), wp, wb, _stream(stream)))


def lava_compact_kv(desc: LayerDesc, k, v, keep_idx, head_offsets, layer_row_offset, k_out, v_out,
                    stream=None) -> None:
    c = desc.to_c()
    _check(load_library().lava_compact_kv(
        ctypes.byref(c), _ptr(k), _ptr(v), _ptr(keep_idx), _ptr(head_offsets),
        _ptr(layer_row_offset), _ptr(k_out), _ptr(v_out), _stream(stream)))


def lava_compact_kv_layers(desc: LayerDesc, n_layers, k, v, k_layer_stride, v_layer_stride,
                           keep_idx, head_offsets, layer_row_offset, k_out, v_out,
                           stream=None) -> None:
    c = desc.to_c()
    _check(load_library().lava_compact_kv_layers(
        ctypes.byref(c), n_layers, _ptr(k), _ptr(v), k_layer_stride, v_layer_stride,
        _ptr(keep_idx), _ptr(head_offsets), _ptr(layer_row_offset), _ptr(k_out), _ptr(v_out),
        _stream(stream)))


# ----------------------------------------------------------------------------- whole model
@dataclass
class EvictionPlan:
    """Device buffers of one full-model eviction (allocated once, reused every step)."""
    desc: LayerDesc
    n_layers: int
    total_budget: torch.Tensor       # int64 [batch]
    floor: torch.Tensor              # int64 [batch]
    cap: torch.Tensor                # int64 [batch]
    scores: torch.Tensor             # float [L, total_scores]
    vbar: torch.Tensor               # float [L, batch, H_kv]
    entropy: torch.Tensor            # double [L, batch]
    layer_budget: torch.Tensor       # int64 [L, batch]
    layer_row_offset: torch.Tensor   # int64 [L*batch + 1]
    keep_idx: torch.Tensor           # int32 [L, total_scores]
    head_offsets: torch.Tensor       # int32 [L, batch, H_kv + 1]
    k_out: torch.Tensor              # [sum of budgets, d]
    v_out: torch.Tensor
    workspace: torch.Tensor          # uint8

    @staticmethod
    def create(desc: LayerDesc, n_layers: int, total_budget, seq_lens, device="cuda",
               kv_dtype=torch.bfloat16) -> "EvictionPlan":
        batch, hkv = desc.batch, desc.n_kv_heads
        i64 = dict(dtype=torch.int64, device=device)
        tb = torch.tensor([int(x) for x in total_budget], **i64)
        floor = torch.tensor([hkv * desc.window] * batch, **i64)
        cap = torch.tensor([hkv * int(n) for n in seq_lens], **i64)
        rows = int(sum(int(x) for x in total_budget))
        ts = desc.total_scores
        ws = torch.zeros(lava_workspace_bytes(desc, n_layers), dtype=torch.uint8, device=device)
        return EvictionPlan(
            desc=desc, n_layers=n_layers, total_budget=tb, floor=floor, cap=cap,
            scores=torch.empty((n_layers, ts), dtype=torch.float32, device=device),
            vbar=torch.empty((n_layers, batch, hkv), dtype=torch.float32, device=device),
            entropy=torch.empty((n_layers, batch), dtype=torch.float64, device=device),
            layer_budget=torch.empty((n_layers, batch), **i64),
            layer_row_offset=torch.empty((n_layers * batch + 1,), **i64),
            keep_idx=torch.empty((n_layers, ts), dtype=torch.int32, device=device),
            head_offsets=torch.empty((n_layers, batch, hkv + 1), dtype=torch.int32, device=device),
            k_out=torch.empty((rows, desc.head_dim), dtype=kv_dtype, device=device),
            v_out=torch.empty((rows, desc.head_dim), dtype=kv_dtype, device=device),
            workspace=ws)


def evict_model(plan: EvictionPlan, q_win, k, v, mode: int = LAVA_BUDGET_DYNAMIC,
                stream=None) -> None:
    """One full-model eviction: score all layers, budgets, layer-wide top-k, compaction.

    q_win [L, batch, H_q, w, d]; k, v [L, H_kv, total_tokens, d] (layer-strided views allowed).
    Four library calls, all enqueued on the current stream; nothing is computed in Python.
    """
    d, nl = plan.desc, plan.n_layers
    lava_score_layers(d, nl, q_win, k, v, q_win.stride(0), k.stride(0), v.stride(0), None,
                      plan.scores, plan.vbar, plan.entropy, plan.workspace, stream)
    lava_layer_budgets(nl, d.batch, plan.entropy, plan.total_budget, plan.floor, plan.cap, mode,
                       plan.layer_budget, plan.layer_row_offset, plan.workspace, stream)
    lava_select_topk_layers(d, nl, plan.scores, plan.layer_budget, plan.keep_idx,
                            plan.head_offsets, plan.workspace, stream)
    lava_compact_kv_layers(d, nl, k, v, k.stride(0), v.stride(0), plan.keep_idx,
                           plan.head_offsets, plan.layer_row_offset, plan.k_out, plan.v_out,
                           stream)


# ----------------------------------------------------------------------------- sharded selection
def lava_select_shard_bytes(desc: LayerDesc, n_layers: int) -> int:
    return load_library().lava_select_shard_bytes(ctypes.byref(desc.to_c()), n_layers)


def lava_select_shard_layout(desc: LayerDesc, n_layers: int):
    """(hist_offset, hist_bytes, ties_offset, ties_bytes) inside the shard state block."""
    v = [ctypes.c_size_t() for _ in range(4)]
    _check(load_library().lava_select_shard_layout(ctypes.byref(desc.to_c()), n_layers,
                                                   *[ctypes.byref(x) for x in v]))
    return tuple(int(x.value) for x in v)


def lava_select_shard_begin(desc, n_layers, total_kv_heads, layer_budget, state, stream=None):
    _check(load_library().lava_select_shard_begin(ctypes.byref(desc.to_c()), n_layers, total_kv_heads,
                                                  _ptr(layer_budget), _ptr(state), state.numel(),
                                                  _stream(stream)))


def lava_select_shard_hist(desc, n_layers, scores, pass_, state, stream=None):
    _check(load_library().lava_select_shard_hist(ctypes.byref(desc.to_c()), n_layers, _ptr(scores),
                                                 pass_, _ptr(state), state.numel(), _stream(stream)))


def lava_select_shard_step(desc, n_layers, pass_, state, stream=None):
    _check(load_library().lava_select_shard_step(ctypes.byref(desc.to_c()), n_layers, pass_,
                                                 _ptr(state), state.numel(), _stream(stream)))


def lava_select_shard_count(desc, n_layers, scores, state, stream=None):
    _check(load_library().lava_select_shard_count(ctypes.byref(desc.to_c()), n_layers, _ptr(scores),
                                                  _ptr(state), state.numel(), _stream(stream)))


def lava_select_shard_emit(desc, n_layers, scores, ties_before_rank, keep_idx, head_offsets,
                           layer_row_offset, state, stream=None):
    _check(load_library().lava_select_shard_emit(
        ctypes.byref(desc.to_c()), n_layers, _ptr(scores), _ptr(ties_before_rank), _ptr(keep_idx),
        _ptr(head_offsets), _ptr(layer_row_offset), _ptr(state), state.numel(), _stream(stream)))


def lava_decode_workspace_bytes(desc: LayerDesc, n_layers: int = 1) -> int:
    return load_library().lava_decode_workspace_bytes(ctypes.byref(desc.to_c()), n_layers)


def lava_decode_attention_layers(desc: LayerDesc, n_layers, q, k_packed, v_packed, head_offsets,
                                 layer_row_offset, out, workspace, stream=None) -> None:
    _check(load_library().lava_decode_attention_layers(
        ctypes.byref(desc.to_c()), n_layers, _ptr(q), _ptr(k_packed), _ptr(v_packed),
        _ptr(head_offsets), _ptr(layer_row_offset), _ptr(out), _ptr(workspace),
        0 if workspace is None else workspace.numel(), _stream(stream)))


def lava_decode_attention(desc: LayerDesc, q, k_packed, v_packed, head_offsets, layer_row_offset,
                          out, workspace, stream=None) -> None:
    _check(load_library().lava_decode_attention(
        ctypes.byref(desc.to_c()), _ptr(q), _ptr(k_packed), _ptr(v_packed), _ptr(head_offsets),
        _ptr(layer_row_offset), _ptr(out), _ptr(workspace),
        0 if workspace is None else workspace.numel(), _stream(stream)))


def lava_layer_output_loss(desc: LayerDesc, q_win, k, v, keep_idx, head_offsets, vbar, w_o,
                           loss_out, bound_out, workspace=None, stream=None):
    """Lemma 1 loss (p = 1, last token) and Theorem 1 bound of one layer's selection."""
    lib = load_library()
    d_model = int(w_o.shape[1])
    need = lib.lava_loss_workspace_bytes(ctypes.byref(desc.to_c()), d_model)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=k.device)
    _check(lib.lava_layer_output_loss(
        ctypes.byref(desc.to_c()), _ptr(q_win), _ptr(k), _ptr(v), _ptr(keep_idx), _ptr(head_offsets),
        _ptr(vbar), _ptr(w_o), _dtype_code(w_o), d_model, _ptr(loss_out), _ptr(bound_out),
        _ptr(workspace), workspace.numel(), _stream(stream)))
    return workspace


# ----------------------------------------------------------------------------- layer by layer
def lava_cascade_state_bytes(desc: LayerDesc, n_layers: int, total_rows: int) -> int:
    n = load_library().lava_cascade_state_bytes(ctypes.byref(desc.to_c()), n_layers, int(total_rows))
    if n == 0:
        raise LavaError(1, "invalid layer descriptor, layer count or row count")
    return n


class Cascade:
    """Algorithm 2, one layer per call (lava_cascade_* of the C ABI).  Owns the device state block
    and a one-layer workspace; `step` takes the layers in order, `view` returns tensors that alias
    the state (valid until the next step)."""

    def __init__(self, desc: LayerDesc, n_layers: int, total_rows: int,
                 mode: int = LAVA_BUDGET_DYNAMIC, device="cuda", kv_dtype=torch.bfloat16):
        self.desc, self.n_layers, self.total_rows, self.kv_dtype = desc, n_layers, int(total_rows), kv_dtype
        self._cdesc = desc.to_c()
        self.state = torch.zeros(lava_cascade_state_bytes(desc, n_layers, total_rows),
                                 dtype=torch.uint8, device=device)
        self.workspace = torch.zeros(lava_workspace_bytes(desc, 1), dtype=torch.uint8, device=device)
        self._h = ctypes.c_void_p()
        _check(load_library().lava_cascade_create(
            ctypes.byref(self._cdesc), n_layers, self.total_rows, mode, _ptr(self.state),
            self.state.numel(), ctypes.byref(self._h)))

    def close(self):
        if self._h:
            load_library().lava_cascade_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def begin(self, total_budget: torch.Tensor, stream=None) -> None:
        _check(load_library().lava_cascade_begin(self._h, _ptr(total_budget), _ptr(self.workspace),
                                                 _stream(stream)))

    def step(self, q_win, k, v, vbar_in=None, stream=None) -> None:
        _check(load_library().lava_cascade_step(self._h, _ptr(q_win), _ptr(k), _ptr(v), _ptr(vbar_in),
                                                _ptr(self.workspace), self.workspace.numel(),
                                                _stream(stream)))

    def view(self) -> dict:
        cv = _CCascadeView()
        _check(load_library().lava_cascade_get(self._h, ctypes.byref(cv)))
        d, done, base = self.desc, cv.layers_done, self.state.data_ptr()

        def at(ptr, nbytes, dtype, shape):
            off = ptr - base
            return self.state[off: off + nbytes].view(dtype).view(shape)

        es = 2 if self.kv_dtype == torch.bfloat16 else 4
        rows, lb = self.total_rows, done * d.batch
        return dict(
            layers_done=done,
            k_out=at(cv.k_out, rows * d.head_dim * es, self.kv_dtype, (rows, d.head_dim)),
            v_out=at(cv.v_out, rows * d.head_dim * es, self.kv_dtype, (rows, d.head_dim)),
            kept_pos=at(cv.kept_pos, rows * 4, torch.int32, (rows,)),
            kept_scores=at(cv.kept_scores, rows * 4, torch.float32, (rows,)),
            head_offsets=at(cv.head_offsets, lb * (d.n_kv_heads + 1) * 4, torch.int32,
                            (done, d.batch, d.n_kv_heads + 1)),
            layer_budget=at(cv.layer_budget, lb * 8, torch.int64, (done, d.batch)),
            layer_row_offset=at(cv.layer_row_offset, (lb + 1) * 8, torch.int64, (lb + 1,)),
            entropy=at(cv.entropy, lb * 8, torch.float64, (done, d.batch)))


# ----------------------------------------------------------------------------- host buffers
def lava_set_option(name: str, value: int) -> None:
    """Process-wide tuning / test knob (see lava.h for the names)."""
    _check(load_library().lava_set_option(name.encode(), int(value)))


def lava_get_option(name: str) -> int:
    v = int(load_library().lava_get_option(name.encode()))
    if v == -(1 << 63):
        raise LavaError(1, lava_last_error())
    return v


def lava_launch_count() -> int:
    return int(load_library().lava_launch_count())


def lava_score_path(desc: LayerDesc) -> int:
    """0 = CUDA-core path, 1 = tensor-core path, 2 = tensor-core path with split query groups."""
    c = desc.to_c()
    r = int(load_library().lava_score_path(ctypes.byref(c)))
    if r < 0:
        raise LavaError(1, load_library().lava_last_error().decode("utf-8", "replace"))
    return r


def lava_host_arena_bytes(desc: LayerDesc, n_layers: int, total_budget_rows: int) -> int:
    c = desc.to_c()
    n = int(load_library().lava_host_arena_bytes(ctypes.byref(c), n_layers, total_budget_rows))
    if n == 0:
        raise LavaError(1, lava_last_error())
    return n


def lava_evict_model_host(desc: LayerDesc, n_layers, q_win, k, v, seq_lens, total_budget, mode,
                          layer_budget, head_offsets, k_out, v_out, arena, stream=None) -> None:
    """All tensor arguments except ``arena`` are HOST tensors (pinned for asynchronous copies);
    seq_lens int32 [batch], total_budget int64 [batch].  Results are complete after the stream
    has been synchronised."""
    c = desc.to_c()
    _check(load_library().lava_evict_model_host(
        ctypes.byref(c), n_layers, _ptr(q_win), _ptr(k), _ptr(v), _ptr(seq_lens),
        _ptr(total_budget), mode, _ptr(layer_budget), _ptr(head_offsets), _ptr(k_out), _ptr(v_out),
        _ptr(arena), arena.numel() * arena.element_size(), _stream(stream)))
