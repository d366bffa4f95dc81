"""ctypes binding of ``libubt.so``: argument marshalling only, every step runs in the CUDA kernels.

The functions carry the names of the C ABI (``include/ubt.h``).  Tensors are ``torch`` CUDA tensors
(device memory and streams are all PyTorch is used for); the host-buffer forms take pinned CPU
tensors.  There is no CPU fallback: a missing library or a non-CUDA tensor raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

from . import _build

UBT_OK = 0
UBT_F32, UBT_BF16 = 0, 1
UBT_VERIFY_GREEDY, UBT_VERIFY_SAMPLE = 0, 1
_MODES = {"greedy": UBT_VERIFY_GREEDY, "sample": UBT_VERIFY_SAMPLE}


class UbtError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class _Tree(C.Structure):
    _fields_ = [("B", C.c_int32), ("N", C.c_int32), ("L", C.c_int32), ("k", C.c_int32), ("mask_words", C.c_int32),
                ("token_ids", C.c_void_p), ("parents", C.c_void_p), ("depths", C.c_void_p),
                ("position_ids", C.c_void_p), ("cand_rank", C.c_void_p), ("scores", C.c_void_p),
                ("mask", C.c_void_p), ("n_nodes", C.c_void_p), ("cand_ids", C.c_void_p),
                ("cand_logprob", C.c_void_p)]


class _DraftOpts(C.Structure):
    _fields_ = [("search_width", C.c_int32), ("depth_bonus", C.c_float), ("alpha", C.c_void_p),
                ("lambda_", C.c_void_p), ("anchor_bigram", C.c_void_p), ("anchor_tokens", C.c_void_p),
                ("pos_offset", C.c_void_p), ("event_between", C.c_void_p), ("status", C.c_void_p),
                ("validate_finite", C.c_int32)]


class _VerifyOpts(C.Structure):
    _fields_ = [("seed", C.c_uint64), ("temperature", C.c_float), ("node_pick", C.c_void_p),
                ("event_before", C.c_void_p), ("event_after", C.c_void_p), ("early_start", C.c_int32),
                ("status", C.c_void_p), ("validate_finite", C.c_int32), ("path_only", C.c_int32)]


class _VerifyResult(C.Structure):
    _fields_ = [("accepted_len", C.c_void_p), ("bonus_token", C.c_void_p), ("accepted_nodes", C.c_void_p),
                ("out_tokens", C.c_void_p)]


EXPORTS = ["ubt_version", "ubt_status_string", "ubt_debug_ring_timeouts", "ubt_draft_workspace_bytes", "ubt_verify_workspace_bytes",
           "ubt_topk_logprob", "ubt_selector_scores", "ubt_build_tree", "ubt_build_mask", "ubt_draft_tree", "ubt_verify_tree",
           "ubt_draft_host_buffer_bytes", "ubt_verify_host_buffer_bytes", "ubt_draft_tree_host",
           "ubt_verify_tree_host", "ubt_verify_tree_static", "ubt_verify_static_capacity", "ubt_lm_head_workspace_bytes",
           "ubt_lm_head_topk", "ubt_topk_shard_bytes", "ubt_topk_shard", "ubt_topk_merge_shards", "ubt_verify_keys_shard",
           "ubt_verify_tree_keys", "ubt_verify_tree_picks", "ubt_sample_totals_shard", "ubt_sample_picks_shard", "ubt_lm_head_topk_shard"]

_lib = None


def lib_path() -> str:
    """``libubt.so`` beside this file; UBT_LIB=checked selects the range-checked debug build."""
    return _build.CHECKED_LIB if os.environ.get("UBT_LIB") == "checked" else _build.LIB


def load() -> C.CDLL:
    """Load ``libubt.so`` (built in-tree by ``_build.build``); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with paper_2609_39972_b200._build.build() "
                          "(needs nvcc); there is no CPU fallback")
    L = C.CDLL(path)
    L.ubt_version.restype = C.c_int
    L.ubt_status_string.restype = C.c_char_p
    L.ubt_status_string.argtypes = [C.c_int]
    for name in ("ubt_draft_workspace_bytes", "ubt_verify_workspace_bytes", "ubt_draft_host_buffer_bytes",
                 "ubt_verify_host_buffer_bytes"):
        getattr(L, name).restype = C.c_size_t
    L.ubt_draft_workspace_bytes.argtypes = [C.c_int] * 5
    L.ubt_verify_workspace_bytes.argtypes = [C.c_int] * 4
    L.ubt_draft_host_buffer_bytes.argtypes = [C.c_int] * 6
    L.ubt_verify_host_buffer_bytes.argtypes = [C.c_int] * 6
    L.ubt_topk_logprob.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                   C.c_void_p, C.c_size_t, C.c_void_p]
    L.ubt_build_tree.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
    L.ubt_build_mask.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
    L.ubt_selector_scores.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
    L.ubt_draft_tree.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                 C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    L.ubt_verify_tree.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                  C.c_void_p, C.c_size_t, C.c_void_p]
    L.ubt_verify_tree_static.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
    L.ubt_verify_static_capacity.restype = C.c_longlong
    L.ubt_lm_head_workspace_bytes.restype = C.c_size_t
    L.ubt_lm_head_workspace_bytes.argtypes = [C.c_int64, C.c_int, C.c_int, C.c_int]
    L.ubt_lm_head_topk.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                   C.c_void_p, C.c_size_t, C.c_void_p]
    L.ubt_lm_head_topk_shard.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int,
                                         C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    L.ubt_topk_shard_bytes.restype = C.c_size_t
    L.ubt_topk_shard_bytes.argtypes = [C.c_int64, C.c_int]
    L.ubt_topk_shard.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                 C.c_size_t, C.c_void_p]
    L.ubt_topk_merge_shards.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
    L.ubt_verify_keys_shard.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                        C.c_size_t, C.c_void_p]
    L.ubt_verify_tree_keys.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
    L.ubt_verify_tree_picks.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
    L.ubt_sample_totals_shard.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int,
                                          C.c_float, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    L.ubt_sample_picks_shard.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                         C.c_int, C.c_uint64, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    L.ubt_debug_ring_timeouts.restype = C.c_longlong
    L.ubt_draft_tree_host.argtypes = L.ubt_draft_tree.argtypes
    L.ubt_verify_tree_host.argtypes = L.ubt_verify_tree.argtypes
    _lib = L
    return L


def ubt_version() -> int:
    return int(load().ubt_version())


def status_string(status: int) -> str:
    return load().ubt_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != UBT_OK:
        raise UbtError(status, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return UBT_BF16
    if t.dtype == torch.float32:
        return UBT_F32
    raise TypeError("logits must be torch.float32 or torch.bfloat16")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _need(t: torch.Tensor, name: str, cuda: bool = True) -> torch.Tensor:
    if cuda and not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (no CPU fallback)")
    if not cuda and t.is_cuda:
        raise ValueError(f"{name} must be a host tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t


def _stream(stream) -> C.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


@dataclass
class Tree:
    """Storage of a batch of draft trees (see ``ubt_tree`` in include/ubt.h)."""
    B: int
    N: int
    L: int
    k: int
    token_ids: torch.Tensor
    parents: torch.Tensor
    depths: torch.Tensor
    position_ids: torch.Tensor
    cand_rank: torch.Tensor
    scores: torch.Tensor
    mask: torch.Tensor
    n_nodes: torch.Tensor
    cand_ids: torch.Tensor
    cand_logprob: torch.Tensor

    @staticmethod
    def empty(B: int, N: int, L: int, k: int, device, pin: bool = False) -> "Tree":
        kw = dict(device=device)
        if pin:
            kw = dict(device="cpu", pin_memory=True)
        i32 = lambda *s: torch.empty(s, dtype=torch.int32, **kw)
        return Tree(B, N, L, k, i32(B, N), i32(B, N), i32(B, N), i32(B, N), i32(B, N),
                    torch.empty((B, N), dtype=torch.float32, **kw), i32(B, N, (N + 31) // 32), i32(B),
                    i32(B, L, k), torch.empty((B, L, k), dtype=torch.float32, **kw))

    def c_struct(self) -> _Tree:
        return _Tree(self.B, self.N, self.L, self.k, (self.N + 31) // 32, self.token_ids.data_ptr(),
                     self.parents.data_ptr(), self.depths.data_ptr(), self.position_ids.data_ptr(),
                     self.cand_rank.data_ptr(), self.scores.data_ptr(), self.mask.data_ptr(),
                     self.n_nodes.data_ptr(), self.cand_ids.data_ptr(), self.cand_logprob.data_ptr())


@dataclass
class VerifyResult:
    accepted_len: torch.Tensor
    bonus_token: torch.Tensor
    accepted_nodes: torch.Tensor
    out_tokens: torch.Tensor
    node_pick: Optional[torch.Tensor] = None

    @staticmethod
    def empty(B: int, L: int, device, pin: bool = False) -> "VerifyResult":
        kw = dict(device="cpu", pin_memory=True) if pin else dict(device=device)
        i32 = lambda *s: torch.empty(s, dtype=torch.int32, **kw)
        return VerifyResult(i32(B), i32(B), i32(B, L + 1), i32(B, L + 1))

    def c_struct(self) -> _VerifyResult:
        return _VerifyResult(self.accepted_len.data_ptr(), self.bonus_token.data_ptr(),
                             self.accepted_nodes.data_ptr(), self.out_tokens.data_ptr())


def _draft_opts(search_width=0, depth_bonus=0.0, alpha=None, lam=None, anchor_bigram=None, anchor_tokens=None,
                pos_offset=None, event_between=None, status=None, validate_finite=False) -> _DraftOpts:
    p = lambda t: None if t is None else t.data_ptr()
    return _DraftOpts(int(search_width), float(depth_bonus), p(alpha), p(lam), p(anchor_bigram), p(anchor_tokens),
                      p(pos_offset), None if event_between is None else event_between.cuda_event, p(status),
                      int(bool(validate_finite)))


def ubt_draft_workspace_bytes(B: int, L: int, V: int, k: int, node_budget: int) -> int:
    return int(load().ubt_draft_workspace_bytes(B, L, V, k, node_budget))


def ubt_verify_workspace_bytes(B: int, node_budget: int, V: int, mode="greedy") -> int:
    return int(load().ubt_verify_workspace_bytes(B, node_budget, V, _MODES.get(mode, mode)))


def workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def ubt_topk_logprob(logits: torch.Tensor, k: int, cand_ids: torch.Tensor, cand_logprob: torch.Tensor,
                     ws: torch.Tensor, stream=None) -> None:
    _need(logits, "logits")
    V = logits.shape[-1]
    rows = logits.numel() // V
    _check(load().ubt_topk_logprob(_ptr(logits), _dtype_code(logits), rows, V, k, _ptr(_need(cand_ids, "cand_ids")),
                                   _ptr(_need(cand_logprob, "cand_logprob")), _ptr(ws), ws.numel(), _stream(stream)),
           "ubt_topk_logprob")


def ubt_topk_shard_bytes(rows: int, k: int) -> int:
    return int(load().ubt_topk_shard_bytes(rows, k))


def ubt_topk_shard(logits_shard: torch.Tensor, k: int, v0: int, partial: Optional[torch.Tensor] = None,
                   ws: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Step a1 on this rank's slice of the vocabulary (columns ``v0 ...`` of every row, dense ``[..., Vs]``):
    returns the rank's per-row partial, a uint8 buffer of ``ubt_topk_shard_bytes(rows, k)`` bytes."""
    _need(logits_shard, "logits_shard")
    Vs = logits_shard.shape[-1]
    rows = logits_shard.numel() // Vs
    if partial is None:
        partial = workspace(ubt_topk_shard_bytes(rows, k), logits_shard.device)
    if ws is None:
        ws = workspace(ubt_draft_workspace_bytes(rows, 1, Vs, k, 1), logits_shard.device)
    _check(load().ubt_topk_shard(_ptr(logits_shard), _dtype_code(logits_shard), rows, Vs, k, int(v0), _ptr(partial),
                                 _ptr(ws), ws.numel(), _stream(stream)), "ubt_topk_shard")
    return partial


def ubt_topk_merge_shards(gathered: torch.Tensor, shards: int, rows: int, k: int,
                          cand_ids: Optional[torch.Tensor] = None, cand_logprob: Optional[torch.Tensor] = None,
                          stream=None):
    """Candidates of the whole rows from the partials of all ranks, back to back in rank order."""
    _need(gathered, "gathered")
    if gathered.numel() * gathered.element_size() < shards * ubt_topk_shard_bytes(rows, k):
        raise ValueError("gathered buffer is smaller than shards * ubt_topk_shard_bytes(rows, k)")
    if cand_ids is None:
        cand_ids = torch.empty((rows, k), dtype=torch.int32, device=gathered.device)
    if cand_logprob is None:
        cand_logprob = torch.empty((rows, k), dtype=torch.float32, device=gathered.device)
    _check(load().ubt_topk_merge_shards(_ptr(gathered), shards, rows, k, _ptr(_need(cand_ids, "cand_ids")),
                                        _ptr(_need(cand_logprob, "cand_logprob")), _stream(stream)),
           "ubt_topk_merge_shards")
    return cand_ids, cand_logprob


def gather_shard_partials(partial: torch.Tensor, group=None) -> tuple:
    """All-gather of the ranks' partials in rank order (NCCL for device buffers): ``(gathered, shards)``.  Without
    an initialised process group the single partial is the gathered buffer."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return partial, 1
    shards = dist.get_world_size(group)
    gathered = torch.empty((shards * partial.numel(),), dtype=partial.dtype, device=partial.device)
    dist.all_gather_into_tensor(gathered, partial.contiguous().view(-1), group=group)
    return gathered, shards


def topk_logprob_vocab_parallel(logits_shard: torch.Tensor, k: int, v0: int, group=None):
    """Step a1 of rows whose vocabulary is split over the ranks of ``group``: local partial, one all-gather,
    merge, all on torch's current stream.  Every rank returns the same ``(cand_ids[rows, k],
    cand_logprob[rows, k])``."""
    Vs = logits_shard.shape[-1]
    rows = logits_shard.numel() // Vs
    partial = ubt_topk_shard(logits_shard, k, v0)
    gathered, shards = gather_shard_partials(partial, group)
    return ubt_topk_merge_shards(gathered, shards, rows, k)


def ubt_lm_head_workspace_bytes(rows: int, d: int, V: int, k: int) -> int:
    return int(load().ubt_lm_head_workspace_bytes(rows, d, V, k))


def ubt_lm_head_topk(hidden: torch.Tensor, weight: torch.Tensor, k: int, cand_ids: Optional[torch.Tensor] = None,
                     cand_logprob: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None, stream=None):
    """LM head fused with step a1: ``hidden[..., d]`` (bf16) x ``weight[V, d]`` (bf16) -> ``(cand_ids[..., k],
    cand_logprob[..., k])``; the logits themselves are never stored."""
    _need(hidden, "hidden"); _need(weight, "weight")
    if hidden.dtype != torch.bfloat16 or weight.dtype != torch.bfloat16:
        raise TypeError("hidden and weight must be torch.bfloat16")
    d = hidden.shape[-1]
    V = weight.shape[0]
    rows = hidden.numel() // d
    if cand_ids is None:
        cand_ids = torch.empty(hidden.shape[:-1] + (k,), dtype=torch.int32, device=hidden.device)
    if cand_logprob is None:
        cand_logprob = torch.empty(hidden.shape[:-1] + (k,), dtype=torch.float32, device=hidden.device)
    if ws is None:
        ws = workspace(ubt_lm_head_workspace_bytes(rows, d, V, k), hidden.device)
    _check(load().ubt_lm_head_topk(_ptr(hidden), _ptr(weight), rows, d, V, k, _ptr(cand_ids), _ptr(cand_logprob),
                                   _ptr(ws), ws.numel(), _stream(stream)), "ubt_lm_head_topk")
    return cand_ids, cand_logprob


def ubt_lm_head_topk_shard(hidden: torch.Tensor, weight_shard: torch.Tensor, k: int, v0: int,
                           partial: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None,
                           stream=None) -> torch.Tensor:
    """The fused LM head on this rank's ``[Vs, d]`` slice of a vocabulary-parallel head (tokens ``v0 ...``): the
    rank's per-row partial (``ubt_topk_shard``'s format); gather and ``ubt_topk_merge_shards`` as for
    ``ubt_topk_shard``."""
    _need(hidden, "hidden"); _need(weight_shard, "weight_shard")
    if hidden.dtype != torch.bfloat16 or weight_shard.dtype != torch.bfloat16:
        raise TypeError("hidden and weight_shard must be torch.bfloat16")
    d = hidden.shape[-1]
    Vs = weight_shard.shape[0]
    rows = hidden.numel() // d
    if partial is None:
        partial = workspace(ubt_topk_shard_bytes(rows, k), hidden.device)
    if ws is None:
        ws = workspace(ubt_lm_head_workspace_bytes(rows, d, Vs, k), hidden.device)
    _check(load().ubt_lm_head_topk_shard(_ptr(hidden), _ptr(weight_shard), rows, d, Vs, k, int(v0), _ptr(partial),
                                         _ptr(ws), ws.numel(), _stream(stream)), "ubt_lm_head_topk_shard")
    return partial


def lm_head_topk_vocab_parallel(hidden: torch.Tensor, weight_shard: torch.Tensor, k: int, v0: int, group=None):
    """LM head + step a1 with the head split along the vocabulary over the ranks of ``group``: fused head on the
    slice, one all-gather of the partials, merge.  Every rank returns the same ``(cand_ids, cand_logprob)``."""
    rows = hidden.numel() // hidden.shape[-1]
    partial = ubt_lm_head_topk_shard(hidden, weight_shard, k, v0)
    gathered, shards = gather_shard_partials(partial, group)
    return ubt_topk_merge_shards(gathered, shards, rows, k)


def ubt_build_tree(bigram_scores: Optional[torch.Tensor], tree: Tree, stream=None, **opts) -> None:
    o = _draft_opts(**opts)
    t = tree.c_struct()
    _check(load().ubt_build_tree(_ptr(bigram_scores), tree.B, tree.L, tree.k, tree.N, C.byref(o), C.byref(t),
                                 _stream(stream)), "ubt_build_tree")


def ubt_selector_scores(phi: torch.Tensor, psi: torch.Tensor, gate: torch.Tensor, cand_ids: torch.Tensor,
                        anchor_tokens: Optional[torch.Tensor] = None, bigram_scores: Optional[torch.Tensor] = None,
                        anchor_bigram: Optional[torch.Tensor] = None, stream=None):
    """Selector scores of all candidate pairs from the codebook tables ``phi``, ``psi`` ``[V,R]`` and the gate
    vectors ``gate[B,L,R]`` (the step between ``ubt_topk_logprob`` and ``ubt_build_tree``).

    Returns ``(bigram_scores[B,L-1,k,k], anchor_bigram[B,k] or None)``.
    """
    for t, n in ((phi, "phi"), (psi, "psi"), (gate, "gate"), (cand_ids, "cand_ids")):
        _need(t, n)
    V, R = phi.shape
    B, L, k = cand_ids.shape
    if bigram_scores is None:
        bigram_scores = torch.empty((B, max(L - 1, 0), k, k), dtype=torch.float32, device=phi.device)
    if anchor_tokens is not None and anchor_bigram is None:
        anchor_bigram = torch.empty((B, k), dtype=torch.float32, device=phi.device)
    _check(load().ubt_selector_scores(_ptr(phi), _ptr(psi), _dtype_code(phi), V, R, _ptr(gate), _ptr(cand_ids),
                                      _ptr(anchor_tokens), B, L, k, _ptr(bigram_scores), _ptr(anchor_bigram),
                                      _stream(stream)), "ubt_selector_scores")
    return bigram_scores, anchor_bigram


def ubt_build_mask(tree: Tree, pos_offset: Optional[torch.Tensor] = None, stream=None) -> None:
    t = tree.c_struct()
    _check(load().ubt_build_mask(C.byref(t), _ptr(pos_offset), _stream(stream)), "ubt_build_mask")


def ubt_draft_tree(unigram_logits: torch.Tensor, bigram_scores: Optional[torch.Tensor], k: int, node_budget: int,
                   tree: Optional[Tree] = None, ws: Optional[torch.Tensor] = None, stream=None, **opts) -> Tree:
    """``unigram_logits[B,L,V]``, ``bigram_scores[B,L-1,k,k]`` -> draft trees (steps a1-a3b)."""
    _need(unigram_logits, "unigram_logits")
    B, L, V = unigram_logits.shape
    if tree is None:
        tree = Tree.empty(B, node_budget, L, k, unigram_logits.device)
    if ws is None:
        ws = workspace(ubt_draft_workspace_bytes(B, L, V, k, node_budget), unigram_logits.device)
    o = _draft_opts(**opts)
    t = tree.c_struct()
    _check(load().ubt_draft_tree(_ptr(unigram_logits), _dtype_code(unigram_logits), _ptr(bigram_scores), B, L, V, k,
                                 node_budget, C.byref(o), C.byref(t), _ptr(ws), ws.numel(), _stream(stream)),
           "ubt_draft_tree")
    return tree


def ubt_verify_tree(tree: Tree, target_logits: torch.Tensor, mode="greedy", seed: int = 0, temperature: float = 1.0,
                    node_pick: Optional[torch.Tensor] = None, result: Optional[VerifyResult] = None,
                    ws: Optional[torch.Tensor] = None, stream=None, event_before=None,
                    event_after=None, early_start: bool = False, status: Optional[torch.Tensor] = None,
                    path_only: bool = False) -> VerifyResult:
    """Walk ``tree`` against ``target_logits[B,N,V]`` (step a4).  ``early_start``, ``path_only``: see
    ``ubt_verify_opts``."""
    _need(target_logits, "target_logits")
    B, N, V = target_logits.shape
    m = _MODES.get(mode, mode)
    if result is None:
        result = VerifyResult.empty(B, tree.L, target_logits.device)
    if ws is None:
        ws = workspace(ubt_verify_workspace_bytes(B, N, V, m), target_logits.device)
    ev = lambda e: None if e is None else C.c_void_p(e.cuda_event)
    o = _VerifyOpts(int(seed), float(temperature), None if node_pick is None else node_pick.data_ptr(),
                    ev(event_before), ev(event_after), int(bool(early_start)),
                    None if status is None else status.data_ptr(), 0, int(bool(path_only)))
    t = tree.c_struct()
    r = result.c_struct()
    _check(load().ubt_verify_tree(C.byref(t), _ptr(target_logits), _dtype_code(target_logits), V, m, C.byref(o),
                                  C.byref(r), _ptr(ws), ws.numel(), _stream(stream)), "ubt_verify_tree")
    result.node_pick = node_pick
    return result


def ubt_verify_keys_shard(target_shard: torch.Tensor, v0: int, row_keys: Optional[torch.Tensor] = None,
                          ws: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Greedy step a4 on this rank's slice of the vocabulary (``target_shard[B, N, Vs]``, first column ``v0``): one
    8-byte ordering key per row, ``int64[B * N]`` (opaque; larger = better pick)."""
    _need(target_shard, "target_shard")
    B, N, Vs = target_shard.shape
    if row_keys is None:
        row_keys = torch.empty((B * N,), dtype=torch.int64, device=target_shard.device)
    if ws is None:
        ws = workspace(ubt_verify_workspace_bytes(B, N, Vs, UBT_VERIFY_GREEDY), target_shard.device)
    _check(load().ubt_verify_keys_shard(_ptr(target_shard), _dtype_code(target_shard), B, N, Vs, int(v0),
                                        _ptr(_need(row_keys, "row_keys")), _ptr(ws), ws.numel(), _stream(stream)),
           "ubt_verify_keys_shard")
    return row_keys


def ubt_verify_tree_keys(tree: Tree, gathered_keys: torch.Tensor, shards: int,
                         node_pick: Optional[torch.Tensor] = None, result: Optional[VerifyResult] = None,
                         status: Optional[torch.Tensor] = None, stream=None) -> VerifyResult:
    """The greedy walk on the ranks' keys, back to back in rank order (``int64[shards * B * N]``)."""
    _need(gathered_keys, "gathered_keys")
    if gathered_keys.numel() < shards * tree.B * tree.N:
        raise ValueError("gathered_keys is smaller than shards * B * N")
    if result is None:
        result = VerifyResult.empty(tree.B, tree.L, gathered_keys.device)
    o = _VerifyOpts(0, 1.0, None if node_pick is None else node_pick.data_ptr(), None, None, 0,
                    None if status is None else status.data_ptr(), 0, 0)
    t = tree.c_struct()
    r = result.c_struct()
    _check(load().ubt_verify_tree_keys(C.byref(t), _ptr(gathered_keys), shards, C.byref(r), C.byref(o),
                                       _stream(stream)), "ubt_verify_tree_keys")
    result.node_pick = node_pick
    return result


def ubt_verify_tree_picks(tree: Tree, node_pick: torch.Tensor, shards: int = 1,
                          result: Optional[VerifyResult] = None, status: Optional[torch.Tensor] = None,
                          stream=None) -> VerifyResult:
    """The walk alone on given per-slot picks ``node_pick`` (``int32[B, N]``, or ``[B * N, 1]`` as
    ``ubt_lm_head_topk`` with ``k = 1`` returns them; with ``shards > 1`` the ranks' picks back to back,
    ``[shards, B, N]``)."""
    _need(node_pick, "node_pick")
    if (node_pick.dtype != torch.int32 or node_pick.numel() != shards * tree.B * tree.N
            or not node_pick.is_contiguous()):
        raise ValueError("node_pick must be a contiguous int32 tensor of shards * B * N entries")
    if result is None:
        result = VerifyResult.empty(tree.B, tree.L, node_pick.device)
    t = tree.c_struct()
    r = result.c_struct()
    _check(load().ubt_verify_tree_picks(C.byref(t), _ptr(node_pick), shards, C.byref(r), _ptr(status),
                                        _stream(stream)), "ubt_verify_tree_picks")
    result.node_pick = node_pick.view(tree.B, tree.N) if shards == 1 else None
    return result


def ubt_sample_totals_shard(target_shard: torch.Tensor, gathered_keys: torch.Tensor, shards: int,
                            temperature: float = 1.0, totals: Optional[torch.Tensor] = None,
                            ws: Optional[torch.Tensor] = None, stream=None):
    """Sampling a4 over a vocabulary-parallel group, second step: the integer weights of this rank's columns summed
    per row (``int64[B * N]``), with the row maximum taken from the gathered keys.  Returns ``(totals, ws)``; pass
    the same ``ws`` to ``ubt_sample_picks_shard``."""
    _need(target_shard, "target_shard"); _need(gathered_keys, "gathered_keys")
    B, N, Vs = target_shard.shape
    if totals is None:
        totals = torch.empty((B * N,), dtype=torch.int64, device=target_shard.device)
    if ws is None:
        ws = workspace(ubt_verify_workspace_bytes(B, N, Vs, "sample"), target_shard.device)
    _check(load().ubt_sample_totals_shard(_ptr(target_shard), _dtype_code(target_shard), B, N, Vs, _ptr(gathered_keys),
                                          shards, float(temperature), _ptr(totals), _ptr(ws), ws.numel(),
                                          _stream(stream)), "ubt_sample_totals_shard")
    return totals, ws


def ubt_sample_picks_shard(target_shard: torch.Tensor, v0: int, rank: int, gathered_totals: torch.Tensor, shards: int,
                           seed: int, ws: torch.Tensor, picks: Optional[torch.Tensor] = None, stream=None):
    """Third step: this rank's picks (``int32[B * N]``: a token where the rank owns the slot's pick, else -1)."""
    _need(target_shard, "target_shard"); _need(gathered_totals, "gathered_totals")
    B, N, Vs = target_shard.shape
    if picks is None:
        picks = torch.empty((B * N,), dtype=torch.int32, device=target_shard.device)
    _check(load().ubt_sample_picks_shard(_ptr(target_shard), _dtype_code(target_shard), B, N, Vs, int(v0), int(rank),
                                         _ptr(gathered_totals), shards, int(seed) & 0xFFFFFFFFFFFFFFFF, _ptr(picks),
                                         _ptr(ws), ws.numel(), _stream(stream)), "ubt_sample_picks_shard")
    return picks


def sample_tree_vocab_parallel(tree: Tree, target_shard: torch.Tensor, v0: int, seed: int, temperature: float = 1.0,
                               group=None, **kw) -> VerifyResult:
    """Sampling verification of target logits whose vocabulary is split over the ranks of ``group`` (ranks in the
    order of their columns): keys, totals and picks with one all-gather each, then the walk; all on torch's current
    stream.  Every rank returns the verdict that one GPU holding whole rows would."""
    import torch.distributed as dist
    rank = dist.get_rank(group) if dist.is_available() and dist.is_initialized() else 0
    keys = ubt_verify_keys_shard(target_shard, v0)
    g_keys, shards = gather_shard_partials(keys, group)
    totals, ws = ubt_sample_totals_shard(target_shard, g_keys, shards, temperature)
    g_tot, _ = gather_shard_partials(totals, group)
    picks = ubt_sample_picks_shard(target_shard, v0, rank, g_tot, shards, seed, ws)
    g_picks, _ = gather_shard_partials(picks, group)
    return ubt_verify_tree_picks(tree, g_picks, shards, **kw)


def verify_tree_from_hidden(tree: Tree, target_hidden: torch.Tensor, weight: torch.Tensor, **kw) -> VerifyResult:
    """Greedy verification from the target's hidden states of the tree slots (``bf16[B, N, d]``) and its LM head
    (``bf16[V, d]``): the head fused with the row arg max (``ubt_lm_head_topk``, k = 1), then the walk; the
    ``[B, N, V]`` target logits are never written to memory."""
    picks, _ = ubt_lm_head_topk(target_hidden.reshape(tree.B * tree.N, -1), weight, 1)
    return ubt_verify_tree_picks(tree, picks, **kw)


def verify_tree_from_hidden_vocab_parallel(tree: Tree, target_hidden: torch.Tensor, weight_shard: torch.Tensor,
                                           v0: int, group=None, **kw) -> VerifyResult:
    """Greedy verification from the target's hidden states with the head split along the vocabulary over the ranks
    of ``group``: fused head + arg max on the slice (k = 1), one all-gather of ``20 B`` per tree slot, merge, walk."""
    picks, _ = lm_head_topk_vocab_parallel(target_hidden.reshape(tree.B * tree.N, -1), weight_shard, 1, v0, group)
    return ubt_verify_tree_picks(tree, picks, **kw)


def verify_tree_vocab_parallel(tree: Tree, target_shard: torch.Tensor, v0: int, group=None, **kw) -> VerifyResult:
    """Greedy verification of target logits whose vocabulary is split over the ranks of ``group``: local keys, one
    all-gather, walk; all on torch's current stream.  Every rank returns the same verdict."""
    keys = ubt_verify_keys_shard(target_shard, v0)
    gathered, shards = gather_shard_partials(keys, group)
    return ubt_verify_tree_keys(tree, gathered, shards, **kw)


def ubt_draft_host_buffer_bytes(B, L, V, k, node_budget, dtype) -> int:
    return int(load().ubt_draft_host_buffer_bytes(B, L, V, k, node_budget, dtype))


def ubt_verify_host_buffer_bytes(B, L, node_budget, V, dtype, mode="greedy") -> int:
    return int(load().ubt_verify_host_buffer_bytes(B, L, node_budget, V, dtype, _MODES.get(mode, mode)))


def ubt_draft_tree_host(unigram_logits: torch.Tensor, bigram_scores: Optional[torch.Tensor], k: int, node_budget: int,
                        tree: Tree, device_buffer: torch.Tensor, stream=None, **opts) -> Tree:
    """Host-buffer form: inputs and ``tree`` live in (pinned) host memory; returns after the stream is idle."""
    _need(unigram_logits, "unigram_logits", cuda=False)
    B, L, V = unigram_logits.shape
    o = _draft_opts(**opts)
    t = tree.c_struct()
    _check(load().ubt_draft_tree_host(_ptr(unigram_logits), _dtype_code(unigram_logits), _ptr(bigram_scores), B, L, V,
                                      k, node_budget, C.byref(o), C.byref(t), _ptr(device_buffer),
                                      device_buffer.numel(), _stream(stream)), "ubt_draft_tree_host")
    return tree


def ubt_verify_tree_host(tree: Tree, target_logits: torch.Tensor, result: VerifyResult, device_buffer: torch.Tensor,
                         mode="greedy", seed: int = 0, temperature: float = 1.0,
                         node_pick: Optional[torch.Tensor] = None, stream=None, status: Optional[torch.Tensor] = None,
                         validate_finite: bool = False) -> VerifyResult:
    _need(target_logits, "target_logits", cuda=False)
    B, N, V = target_logits.shape
    o = _VerifyOpts(int(seed), float(temperature), None if node_pick is None else node_pick.data_ptr(), None, None, 0,
                    None if status is None else status.data_ptr(), int(bool(validate_finite)), 0)
    t = tree.c_struct()
    r = result.c_struct()
    _check(load().ubt_verify_tree_host(C.byref(t), _ptr(target_logits), _dtype_code(target_logits), V,
                                       _MODES.get(mode, mode), C.byref(o), C.byref(r), _ptr(device_buffer),
                                       device_buffer.numel(), _stream(stream)), "ubt_verify_tree_host")
    result.node_pick = node_pick
    return result


def ubt_verify_static_capacity() -> int:
    """Keys (one per target row and span) the built-in scratch of ``ubt_verify_tree_static`` holds."""
    return int(load().ubt_verify_static_capacity())


def ubt_verify_tree_static(tree: Tree, target_logits: torch.Tensor, node_pick: Optional[torch.Tensor] = None,
                           result: Optional[VerifyResult] = None, stream=None) -> VerifyResult:
    """Greedy ``ubt_verify_tree`` for callers that cannot allocate device memory.

    The library call takes no workspace and allocates nothing: its scratch is a fixed 512 KiB array inside
    ``libubt.so``.  Pass ``result`` (and ``node_pick``) preallocated if this wrapper, too, must not allocate.
    Calls share that one array, so calls that may overlap on the GPU have to be serialised by the caller.
    """
    _need(target_logits, "target_logits")
    B, N, V = target_logits.shape
    if result is None:
        result = VerifyResult.empty(B, tree.L, target_logits.device)
    t = tree.c_struct()
    r = result.c_struct()
    _check(load().ubt_verify_tree_static(C.byref(t), _ptr(target_logits), _dtype_code(target_logits), V,
                                         _ptr(node_pick), C.byref(r), _stream(stream)), "ubt_verify_tree_static")
    result.node_pick = node_pick
    return result


def ubt_debug_ring_timeouts() -> int:
    """Bounded device-side waits that gave up since the library was loaded (0 in a healthy process)."""
    return int(load().ubt_debug_ring_timeouts())
