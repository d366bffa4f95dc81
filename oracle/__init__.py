"""Python face of the CPU oracle (test infrastructure, never the product path).

Compiles ``ubt_oracle.c`` with gcc on first use and exposes its functions with
numpy arrays.  Only tests, the smoke check and the benchmark's CPU-baseline leg
may import this package; the CUDA library and its binding never do.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ubt_oracle.c")
_LIB = os.path.join(_HERE, "libubt_oracle.so")
_lib = None

F32, BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle into ``oracle/libubt_oracle.so`` (gcc, -O2, no fp contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=gnu11", "-ffp-contract=off", "-fopenmp", "-shared",
                               "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.ubt_oracle_weight.restype = C.c_uint64
        _lib.ubt_oracle_weight.argtypes = [C.c_float, C.c_float, C.c_float]
        _lib.ubt_oracle_row_cdf.restype = C.c_uint64
        _lib.ubt_oracle_row_cdf.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int, C.c_float, C.c_void_p]
        _lib.ubt_oracle_threshold.restype = C.c_uint64
        _lib.ubt_oracle_threshold.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64]
        _lib.ubt_oracle_topk_logprob.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int, C.c_int,
                                                 C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.ubt_oracle_build_tree.argtypes = (
            [C.c_void_p] * 3 + [C.c_int] * 5 + [C.c_double] + [C.c_void_p] * 15)
        _lib.ubt_oracle_verify.argtypes = (
            [C.c_void_p] * 3 + [C.c_int] * 3 + [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_uint64,
                                                C.c_float] + [C.c_void_p] * 5)
        _lib.ubt_oracle_walks_from_cdf.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p,
                                                   C.c_uint32, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        _lib.ubt_oracle_weight_consts.argtypes = [C.c_float, C.c_float, C.c_void_p, C.c_void_p]
        _lib.ubt_oracle_walk_picks.argtypes = [C.c_void_p] * 3 + [C.c_int] * 3 + [C.c_void_p] * 5
        _lib.ubt_oracle_lm_head_topk.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_int, C.c_int, C.c_int,
                                                 C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.ubt_oracle_selector_scores.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_int, C.c_void_p,
                                                    C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                                    C.c_void_p]
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.uint16:
        return BF16
    if a.dtype == np.float32:
        return F32
    raise TypeError("logits must be float32 or uint16 (bf16 bit patterns)")


def num_threads() -> int:
    return int(lib().ubt_oracle_num_threads())


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, np.uint32).copy()
    k = np.asarray(key, np.uint32).copy()
    out = np.zeros(4, np.uint32)
    lib().ubt_oracle_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def topk_logprob(logits: np.ndarray, k: int):
    """Step 1 on ``logits[..., V]`` -> (cand_ids[..., k] i32, cand_lp[..., k] f64, lse[...] f64)."""
    logits = np.ascontiguousarray(logits)
    V = logits.shape[-1]
    rows = int(np.prod(logits.shape[:-1], dtype=np.int64))
    ids = np.empty(logits.shape[:-1] + (k,), np.int32)
    lp = np.empty(logits.shape[:-1] + (k,), np.float64)
    lse = np.empty(logits.shape[:-1], np.float64)
    rc = lib().ubt_oracle_topk_logprob(_p(logits), _dtype_code(logits), rows, V, k, _p(ids), _p(lp), _p(lse))
    if rc:
        raise ValueError("oracle topk_logprob rejected its arguments")
    return ids, lp, lse


def lm_head_topk(hidden: np.ndarray, weight: np.ndarray, k: int, want_logits: bool = False):
    """Unigram logits ``hidden[rows, d] @ weight[V, d].T`` in double, then step 1 on them (Section 3.1.1, eq. 3).

    ``hidden`` and ``weight`` are fp32, or bf16 bit patterns as uint16.  Returns ``(cand_ids[rows, k] i32,
    cand_lp[rows, k] f64, lse[rows] f64, logits[rows, V] f64 or None)``.
    """
    hidden = np.ascontiguousarray(hidden); weight = np.ascontiguousarray(weight)
    rows, d = hidden.shape
    V, d2 = weight.shape
    assert d == d2 and hidden.dtype == weight.dtype
    ids = np.empty((rows, k), np.int32)
    lp = np.empty((rows, k), np.float64)
    lse = np.empty(rows, np.float64)
    logits = np.empty((rows, V), np.float64) if want_logits else None
    rc = lib().ubt_oracle_lm_head_topk(_p(hidden), _p(weight), _dtype_code(hidden), rows, d, V, k, _p(ids), _p(lp),
                                       _p(lse), _p(logits) if want_logits else None)
    if rc:
        raise ValueError("oracle lm_head_topk rejected its arguments")
    return ids, lp, lse, logits


def selector_scores(phi: np.ndarray, psi: np.ndarray, gate: np.ndarray, cand_ids: np.ndarray,
                    anchor_tokens: Optional[np.ndarray] = None):
    """Selector scores of all candidate pairs (Section 3.1.2, "Parallel Computation").

    ``phi``, ``psi``: codebook tables ``[V, R]`` (fp32, or bf16 bit patterns as uint16); ``gate[B, L, R]`` fp32 is
    the projected proposer state of each position; ``cand_ids[B, L, k]``.  Returns ``(bigram[B, L-1, k, k] f64,
    anchor_bigram[B, k] f64 or None)``.
    """
    phi = np.ascontiguousarray(phi); psi = np.ascontiguousarray(psi)
    gate = np.ascontiguousarray(gate, np.float32); cand_ids = np.ascontiguousarray(cand_ids, np.int32)
    V, R = phi.shape
    B, L, k = cand_ids.shape
    assert psi.shape == (V, R) and gate.shape == (B, L, R) and phi.dtype == psi.dtype
    big = np.zeros((B, max(L - 1, 0), k, k), np.float64)
    anc = None
    if anchor_tokens is not None:
        anchor_tokens = np.ascontiguousarray(anchor_tokens, np.int32)
        anc = np.zeros((B, k), np.float64)
    rc = lib().ubt_oracle_selector_scores(_p(phi), _p(psi), _dtype_code(phi), V, R, _p(gate), _p(cand_ids),
                                          _p(anchor_tokens) if anchor_tokens is not None else None, B, L, k,
                                          _p(big), _p(anc) if anc is not None else None)
    if rc:
        raise ValueError("oracle selector_scores rejected its arguments")
    return big, anc


@dataclass
class Tree:
    token_ids: np.ndarray     # [B,N] i32
    parents: np.ndarray       # [B,N] i32
    depths: np.ndarray        # [B,N] i32
    cand_rank: np.ndarray     # [B,N] i32
    position_ids: np.ndarray  # [B,N] i32
    scores: np.ndarray        # [B,N] f64
    mask: np.ndarray          # [B,N,ceil(N/32)] u32
    n_nodes: np.ndarray       # [B] i32
    t: np.ndarray             # [B,L,k,k] f64  log q^bi
    min_cut_gap: np.ndarray   # [B] f64
    cand_ids: Optional[np.ndarray] = None
    cand_lp: Optional[np.ndarray] = None


def build_tree(cand_ids, cand_lp, bigram, N: int, W: int = 0, zeta: float = 0.0, alpha=None, lam=None,
               anchor_bigram=None, anchor_tokens=None, pos_offset=None) -> Tree:
    """Steps 2-3 (Algorithm 1) from candidates and bigram scores."""
    cand_ids = np.ascontiguousarray(cand_ids, np.int32)
    cand_lp = np.ascontiguousarray(cand_lp, np.float64)
    B, L, k = cand_ids.shape
    bigram = np.ascontiguousarray(bigram, np.float32)
    assert bigram.shape == (B, max(L - 1, 0), k, k), bigram.shape
    f32 = lambda a: None if a is None else np.ascontiguousarray(a, np.float32)
    i32 = lambda a: None if a is None else np.ascontiguousarray(a, np.int32)
    alpha, lam, anchor_bigram = f32(alpha), f32(lam), f32(anchor_bigram)
    anchor_tokens, pos_offset = i32(anchor_tokens), i32(pos_offset)
    mw = (N + 31) // 32
    tr = Tree(*(np.empty((B, N), np.int32) for _ in range(5)), np.empty((B, N), np.float64),
              np.empty((B, N, mw), np.uint32), np.empty(B, np.int32), np.empty((B, L, k, k), np.float64),
              np.empty(B, np.float64), cand_ids, cand_lp)
    rc = lib().ubt_oracle_build_tree(
        _p(cand_ids), _p(cand_lp), _p(bigram), B, L, k, N, W, float(zeta), _p(alpha), _p(lam),
        _p(anchor_bigram), _p(anchor_tokens), _p(pos_offset), _p(tr.token_ids), _p(tr.parents),
        _p(tr.depths), _p(tr.cand_rank), _p(tr.position_ids), _p(tr.scores), _p(tr.mask), _p(tr.n_nodes),
        _p(tr.t), _p(tr.min_cut_gap))
    if rc:
        raise ValueError("oracle build_tree failed (bad arguments or a selection that is not prefix-closed)")
    return tr


def draft_tree(unigram_logits, bigram, k: int, N: int, **kw) -> Tree:
    """Steps 1-3: ``unigram_logits[B,L,V]``, ``bigram[B,L-1,k,k]`` -> Tree."""
    ids, lp, _ = topk_logprob(unigram_logits, k)
    return build_tree(ids, lp, bigram, N, **kw)


@dataclass
class Verdict:
    accepted_len: np.ndarray    # [B]
    accepted_nodes: np.ndarray  # [B,L+1]
    out_tokens: np.ndarray      # [B,L+1]
    bonus_token: np.ndarray     # [B]
    node_pick: Optional[np.ndarray]  # [B,N] or None


def verify(token_ids, parents, n_nodes, L: int, target_logits, mode: str = "greedy", seed: int = 0,
           temperature: float = 1.0, all_nodes: bool = True) -> Verdict:
    """Step 4 on a tree given by its arrays; ``all_nodes`` also evaluates unused rows."""
    token_ids = np.ascontiguousarray(token_ids, np.int32)
    parents = np.ascontiguousarray(parents, np.int32)
    n_nodes = np.ascontiguousarray(n_nodes, np.int32)
    z = np.ascontiguousarray(target_logits)
    B, N, V = z.shape
    assert token_ids.shape == (B, N)
    out = Verdict(np.empty(B, np.int32), np.empty((B, L + 1), np.int32), np.empty((B, L + 1), np.int32),
                  np.empty(B, np.int32), np.empty((B, N), np.int32) if all_nodes else None)
    rc = lib().ubt_oracle_verify(_p(token_ids), _p(parents), _p(n_nodes), B, N, L, _p(z), _dtype_code(z), V,
                                 {"greedy": 0, "sample": 1}[mode], int(seed), float(temperature),
                                 _p(out.accepted_len), _p(out.accepted_nodes), _p(out.out_tokens),
                                 _p(out.bonus_token), _p(out.node_pick))
    if rc:
        raise ValueError("oracle verify rejected its arguments")
    return out


def verify_picks(token_ids, parents, n_nodes, L: int, picks) -> Verdict:
    """The walk of step 4 alone on given per-slot picks ``picks[B,N]`` (Appendix A, verification)."""
    token_ids = np.ascontiguousarray(token_ids, np.int32)
    parents = np.ascontiguousarray(parents, np.int32)
    n_nodes = np.ascontiguousarray(n_nodes, np.int32)
    picks = np.ascontiguousarray(picks, np.int32)
    B, N = token_ids.shape
    assert picks.shape == (B, N)
    out = Verdict(np.empty(B, np.int32), np.empty((B, L + 1), np.int32), np.empty((B, L + 1), np.int32),
                  np.empty(B, np.int32), picks)
    rc = lib().ubt_oracle_walk_picks(_p(token_ids), _p(parents), _p(n_nodes), B, N, L, _p(picks),
                                     _p(out.accepted_len), _p(out.accepted_nodes), _p(out.out_tokens),
                                     _p(out.bonus_token))
    if rc:
        raise ValueError("oracle walk rejected its arguments")
    return out


def row_cdf(target_logits: np.ndarray, row: int, temperature: float = 1.0) -> np.ndarray:
    """Inclusive prefix sums (u64) of the integer sampling weights of one row."""
    z = np.ascontiguousarray(target_logits)
    V = z.shape[-1]
    pre = np.empty(V, np.uint64)
    lib().ubt_oracle_row_cdf(_p(z), _dtype_code(z), int(row), V, float(temperature), _p(pre))
    return pre


def weight(z: float, a: float, c: float) -> int:
    return int(lib().ubt_oracle_weight(z, a, c))


def weight_consts(row_max: float, temperature: float):
    a, c = C.c_float(), C.c_float()
    lib().ubt_oracle_weight_consts(row_max, temperature, C.byref(a), C.byref(c))
    return a.value, c.value


def threshold(seed: int, b: int, n: int, total: int) -> int:
    return int(lib().ubt_oracle_threshold(seed, b, n, total))


def walks_from_cdf(token_ids, parents, n_nodes: int, cdf: np.ndarray, b: int, seeds: np.ndarray):
    """Sampling walks of one sequence for many seeds, from per-row CDFs ``cdf[N,V]``."""
    token_ids = np.ascontiguousarray(token_ids, np.int32)
    parents = np.ascontiguousarray(parents, np.int32)
    cdf = np.ascontiguousarray(cdf, np.uint64)
    seeds = np.ascontiguousarray(seeds, np.uint64)
    acc = np.empty(len(seeds), np.int32)
    bonus = np.empty(len(seeds), np.int32)
    lib().ubt_oracle_walks_from_cdf(_p(token_ids), _p(parents), int(n_nodes), cdf.shape[1], _p(cdf), int(b),
                                    _p(seeds), len(seeds), _p(acc), _p(bonus))
    return acc, bonus
