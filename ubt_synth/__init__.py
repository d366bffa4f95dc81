"""Seeded synthetic inputs for the UBTree draft+verify hot path.

This module only draws random numbers and lays them out; it holds none of the
method's arithmetic (no softmax, no top-k, no tree logic).  Both the CPU oracle
and the CUDA path are fed the *same bytes* produced here.

The paper measures on GSM8K, MATH-500, AIME, HumanEval, MBPP, LiveCodeBench,
MT-Bench, LongBench-v2 and SWE-bench with trained Qwen3 / Ling drafters
(Section 4, Table 1).  None of those datasets or weights is needed by this
path, which consumes logits only; the generators below stand in for them with
the Qwen3 vocabulary size (V = 151,936), the paper's block and budget sizes and
an entropy spread (logit scale s) that covers near-deterministic to flat rows.

bf16 tensors are carried on the host as ``uint16`` bit patterns (numpy has no
bf16); :func:`f32_to_bf16_bits` rounds to nearest-even exactly as a hardware
conversion does.

Two backends draw the noise:
  * ``numpy``  -- ``numpy.random.Generator(PCG64)``, one child stream per
    (tensor, batch index) via ``SeedSequence.spawn``; canonical, used by tests.
  * ``torch``  -- a seeded ``torch.Generator`` on a CUDA device, for the
    multi-GB bench tensors; the values differ from the numpy backend but are
    a deterministic function of the seed on a given device type.
"""
from __future__ import annotations

import dataclasses
import math
from concurrent.futures import ThreadPoolExecutor
from typing import Optional

import numpy as np

V_QWEN3 = 151_936


@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    B: int
    L: int
    V: int
    k: int
    N: int                 # node budget: tree slots INCLUDING the root
    dtype: str             # "f32" | "bf16"
    scale: str             # recipe for the per-row logit scale s
    bigram_std: float
    spike: float           # added to one token per draft position (0 = none)
    mode: str              # "greedy" | "sample"

    def replace(self, **kw) -> "Config":
        return dataclasses.replace(self, **kw)


CONFIGS = {
    # Tiny exactness case (fp32).
    "c1": Config("c1", 1, 4, 1000, 4, 16, "f32", "fixed:0.5,2,6,2", 1.0, 0.0, "greedy"),
    # Qwen3-8B-shaped single stream.
    "c2": Config("c2", 1, 16, V_QWEN3, 8, 64, "bf16", "pos_uniform:0.5,8", 1.0, 4.0, "greedy"),
    # Batched serving, per-sequence entropy log-uniform.
    "c3": Config("c3", 32, 16, V_QWEN3, 8, 64, "bf16", "seq_loguniform:0.3,10", 1.5, 0.0, "greedy"),
    # Wide tree, high entropy.
    "c4": Config("c4", 64, 32, V_QWEN3, 16, 256, "bf16", "pos_uniform:0.3,2", 2.0, 0.0, "greedy"),
    # Sampling verify at scale.
    "c5": Config("c5", 128, 16, V_QWEN3, 8, 128, "bf16", "pos_uniform:0.5,4", 1.0, 0.0, "sample"),
}


# The paper's own search configuration (Appendix B, "Training and Inference Configuration"): K = 64 candidates,
# search width 12, 64 non-root nodes, 15 future positions, selector rank 256; run through the split entry points
# with the selector scores computed on the device.  B = 32 concurrent streams, as in the serving experiments.
SELECTOR_RANK = 256
PAPER_SEARCH_WIDTH = 12
NEXT_CONFIGS = {
    "p1": Config("p1", 32, 15, V_QWEN3, 64, 65, "bf16", "pos_uniform:0.5,8", 1.0, 4.0, "greedy"),
    "p1-b1": Config("p1-b1", 1, 15, V_QWEN3, 64, 65, "bf16", "pos_uniform:0.5,8", 1.0, 4.0, "greedy"),
    # The smaller (budget / width) pairs of the paper's load-adaptive serving setup ("Academic-scale
    # Experiment", concurrent serving): 32 / 8 and 16 / 3 non-root nodes / search width.
    "p2": Config("p2", 32, 15, V_QWEN3, 64, 33, "bf16", "pos_uniform:0.5,8", 1.0, 4.0, "greedy"),
    "p3": Config("p3", 32, 15, V_QWEN3, 64, 17, "bf16", "pos_uniform:0.5,8", 1.0, 4.0, "greedy"),
}
SEARCH_WIDTH = {"p1": 12, "p1-b1": 12, "p2": 8, "p3": 3}


def search_width(cfg: "Config") -> int:
    """Search width the paper pairs with a next-row configuration (0 = unbounded for the others)."""
    return SEARCH_WIDTH.get(cfg.name.split("-B")[0], 0)


# --------------------------------------------------------------------------
# bf16 helpers (bit-level, no arithmetic of the method)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 -> bf16 (nearest, ties to even); returns uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    out = ((u + rounding) >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen uint16 bf16 bit patterns to fp32 (exact)."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def as_f32(values: np.ndarray, dtype: str) -> np.ndarray:
    """fp32 view of a host tensor produced by this module."""
    return bf16_bits_to_f32(values) if dtype == "bf16" else np.asarray(values, np.float32)


# --------------------------------------------------------------------------
# scales
# --------------------------------------------------------------------------
def _row_scales(recipe: str, rng: np.random.Generator, B: int, rows: int) -> np.ndarray:
    """Scale s for each of [B, rows] logit rows according to the recipe string."""
    kind, _, args = recipe.partition(":")
    a = [float(t) for t in args.split(",")]
    if kind == "fixed":
        s = np.array([a[i % len(a)] for i in range(rows)], np.float64)
        return np.broadcast_to(s, (B, rows)).copy()
    if kind == "pos_uniform":
        return rng.uniform(a[0], a[1], size=(B, rows))
    if kind == "seq_loguniform":
        s = np.exp(rng.uniform(math.log(a[0]), math.log(a[1]), size=(B, 1)))
        return np.broadcast_to(s, (B, rows)).copy()
    raise ValueError(f"unknown scale recipe {recipe!r}")


def _fill_rows_numpy(out: np.ndarray, scales: np.ndarray, seeds, dtype: str,
                     threads: int = 8) -> None:
    """out[b] <- dtype(N(0,1) * scales[b, row]) with one child stream per b."""
    B = out.shape[0]

    def work(b: int) -> None:
        rng = np.random.Generator(np.random.PCG64(seeds[b]))
        rows, V = out.shape[1], out.shape[2]
        step = max(1, (1 << 24) // V)
        for r0 in range(0, rows, step):
            r1 = min(rows, r0 + step)
            z = rng.standard_normal((r1 - r0, V), dtype=np.float32)
            z *= scales[b, r0:r1, None].astype(np.float32)
            out[b, r0:r1] = f32_to_bf16_bits(z) if dtype == "bf16" else z

    if B == 1 or threads <= 1:
        for b in range(B):
            work(b)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(work, range(B)))


def _empty(shape, dtype: str) -> np.ndarray:
    return np.empty(shape, np.uint16 if dtype == "bf16" else np.float32)


# --------------------------------------------------------------------------
# public generators (numpy backend)
# --------------------------------------------------------------------------
@dataclasses.dataclass
class DraftInputs:
    cfg: Config
    unigram_logits: np.ndarray      # [B,L,V] float32, or uint16 bf16 bits
    bigram_scores: np.ndarray       # [B,L-1,k,k] float32
    scales: np.ndarray              # [B,L] the s used per row (for the record)


def draft_inputs(cfg: Config, seed: int = 0) -> DraftInputs:
    """Unigram block logits and bigram transition scores for one batch."""
    ss = np.random.SeedSequence([seed, 0xD4AF7])
    s_meta, s_big, s_spike, *s_rows = ss.spawn(3 + cfg.B)
    meta = np.random.Generator(np.random.PCG64(s_meta))
    scales = _row_scales(cfg.scale, meta, cfg.B, cfg.L)
    u = _empty((cfg.B, cfg.L, cfg.V), cfg.dtype)
    _fill_rows_numpy(u, scales, s_rows, cfg.dtype)
    if cfg.spike:
        rs = np.random.Generator(np.random.PCG64(s_spike))
        tok = rs.integers(0, cfg.V, size=(cfg.B, cfg.L))
        bi, li = np.meshgrid(np.arange(cfg.B), np.arange(cfg.L), indexing="ij")
        if cfg.dtype == "bf16":
            v = bf16_bits_to_f32(u[bi, li, tok]) + np.float32(cfg.spike)
            u[bi, li, tok] = f32_to_bf16_bits(v)
        else:
            u[bi, li, tok] += np.float32(cfg.spike)
    rb = np.random.Generator(np.random.PCG64(s_big))
    big = (rb.standard_normal((cfg.B, max(cfg.L - 1, 0), cfg.k, cfg.k), dtype=np.float32)
           * np.float32(cfg.bigram_std))
    return DraftInputs(cfg, u, np.ascontiguousarray(big), scales)


def target_logits(cfg: Config, seed: int = 0) -> np.ndarray:
    """Target-model logits [B,N,V] drawn from the same recipe as the draft rows."""
    ss = np.random.SeedSequence([seed, 0x7A26E7])
    s_meta, *s_rows = ss.spawn(1 + cfg.B)
    meta = np.random.Generator(np.random.PCG64(s_meta))
    scales = _row_scales(cfg.scale, meta, cfg.B, cfg.N)
    z = _empty((cfg.B, cfg.N, cfg.V), cfg.dtype)
    _fill_rows_numpy(z, scales, s_rows, cfg.dtype)
    return z


def _set(z: np.ndarray, dtype: str, idx, value: np.ndarray) -> None:
    if dtype == "bf16":
        z[idx] = f32_to_bf16_bits(np.asarray(value, np.float32).reshape(1))[0]
    else:
        z[idx] = np.asarray(value, np.float32)


def plant_path(z: np.ndarray, dtype: str, token_ids: np.ndarray, parents: np.ndarray,
               n_nodes: np.ndarray, seed: int = 0, boost: float = 1.0) -> np.ndarray:
    """Plant a random root-to-node path as the row maxima of target logits.

    For each sequence pick a random node of its tree; on every node of the path
    root -> that node (excluding the end node) raise the logit of the next path
    token to ``rowmax + boost``.  At the end node raise a token that is not one
    of its children's tokens, so a greedy walk stops exactly there.  Returns the
    planted end node per sequence (its depth is the expected accepted length).
    Only indexing and a row maximum are used here: the tree is an input.
    """
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 0x91A27])))
    B, N, V = z.shape
    ends = np.zeros(B, np.int64)
    for b in range(B):
        n = int(n_nodes[b])
        end = int(rng.integers(0, n))
        ends[b] = end
        path = [end]
        while parents[b, path[-1]] >= 0:
            path.append(int(parents[b, path[-1]]))
        path.reverse()                      # root ... end
        for a, c in zip(path[:-1], path[1:]):
            top = as_f32(z[b, a], dtype).max()
            _set(z, dtype, (b, a, int(token_ids[b, c])), top + np.float32(boost))
        kids = {int(token_ids[b, c]) for c in range(n) if parents[b, c] == end}
        stop_tok = int(rng.integers(0, V))
        while stop_tok in kids:
            stop_tok = (stop_tok + 1) % V
        top = as_f32(z[b, end], dtype).max()
        _set(z, dtype, (b, end, stop_tok), top + np.float32(boost))
    return ends


def agree_targets(cfg: Config, unigram_logits: np.ndarray, token_ids: np.ndarray,
                  parents: np.ndarray, depths: np.ndarray, n_nodes: np.ndarray,
                  seed: int = 0, noise_std: float = 0.5) -> np.ndarray:
    """Targets that resemble the drafter, so acceptance lengths are realistic.

    The row of a node at depth d is ``u[b, d, :] + N(0, noise_std^2)`` (the
    drafter approximates the target; depth-L nodes reuse position L-1) and one
    randomly chosen child of each node gets ``+g``, g ~ U[2, 8], on its token.
    Unused slots (>= n_nodes) are plain noise.
    """
    ss = np.random.SeedSequence([seed, 0xA62EE])
    B, N, V, L = cfg.B, cfg.N, cfg.V, cfg.L
    z = _empty((B, N, V), cfg.dtype)
    children = ss.spawn(B)
    for b in range(B):
        rng = np.random.Generator(np.random.PCG64(children[b]))
        for n in range(N):
            noise = rng.standard_normal(V, dtype=np.float32) * np.float32(noise_std)
            if n < n_nodes[b]:
                d = min(int(depths[b, n]), L - 1)
                row = as_f32(unigram_logits[b, d], cfg.dtype) + noise
                kids = [c for c in range(int(n_nodes[b])) if parents[b, c] == n]
                if kids:
                    c = kids[int(rng.integers(0, len(kids)))]
                    row[int(token_ids[b, c])] += np.float32(rng.uniform(2.0, 8.0))
            else:
                row = noise
            z[b, n] = f32_to_bf16_bits(row) if cfg.dtype == "bf16" else row
    return z


# --------------------------------------------------------------------------
# torch backend: bulk noise drawn on a CUDA device (bench-sized tensors)
# --------------------------------------------------------------------------
def device_inputs(cfg: Config, seed: int, device, want_target: bool = True):
    """Same recipes as above, drawn with a seeded torch generator on ``device``.

    Returns ``(unigram_logits, bigram_scores, target_logits)`` as torch tensors
    (bf16 or fp32 per the config) resident on ``device``.
    """
    import torch

    g = torch.Generator(device=device)
    g.manual_seed(int(seed) * 1_000_003 + 0x5EED)
    meta = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 0x70C4])))
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32

    def rows(nrows: int) -> "torch.Tensor":
        s = torch.from_numpy(_row_scales(cfg.scale, meta, cfg.B, nrows).astype(np.float32)).to(device)
        out = torch.empty((cfg.B, nrows, cfg.V), dtype=tdt, device=device)
        step = max(1, (1 << 28) // (nrows * cfg.V))
        for b0 in range(0, cfg.B, step):
            b1 = min(cfg.B, b0 + step)
            z = torch.randn((b1 - b0, nrows, cfg.V), generator=g, device=device, dtype=torch.float32)
            z.mul_(s[b0:b1, :, None])
            out[b0:b1] = z.to(tdt)
        return out

    u = rows(cfg.L)
    if cfg.spike:
        tok = torch.from_numpy(meta.integers(0, cfg.V, size=(cfg.B, cfg.L))).to(device)
        cur = torch.gather(u.float(), 2, tok[..., None]) + cfg.spike
        u.scatter_(2, tok[..., None], cur.to(tdt))
    big = torch.randn((cfg.B, max(cfg.L - 1, 0), cfg.k, cfg.k), generator=g, device=device,
                      dtype=torch.float32) * cfg.bigram_std
    z = rows(cfg.N) if want_target else None
    return u, big.contiguous(), z


def selector_tables(V: int, R: int, B: int, L: int, seed: int, dtype: str = "bf16"):
    """Synthetic stand-ins for the selector's precomputed codebook tables and gate vectors.

    Returns ``(phi[V,R], psi[V,R], gate[B,L,R] fp32)``; tables are N(0,1) in the given dtype (bf16 as bit
    patterns), gates N(0, 1/R), so that a pair score, a sum of R products, has unit scale like the
    configurations' bigram scores.
    """
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 0x5E1EC7])))
    phi = rng.standard_normal((V, R), dtype=np.float32)
    psi = rng.standard_normal((V, R), dtype=np.float32)
    gate = (rng.standard_normal((B, L, R), dtype=np.float32) / np.sqrt(np.float32(R))).astype(np.float32)
    if dtype == "bf16":
        phi, psi = f32_to_bf16_bits(phi), f32_to_bf16_bits(psi)
    return phi, psi, gate


def lm_head_inputs(rows: int, d: int, V: int, seed: int, scale: float = 2.0, dtype: str = "bf16"):
    """Synthetic stand-ins for the proposer's hidden states and the frozen LM head: ``hidden[rows, d]`` N(0,1) and
    ``weight[V, d]`` N(0, scale^2 / d), so that a logit (a sum of d products) is N(0, scale^2) like the
    configurations' unigram logits.  bf16 as bit patterns (uint16), or fp32."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 0x11EAD])))
    h = rng.standard_normal((rows, d), dtype=np.float32)
    w = (rng.standard_normal((V, d), dtype=np.float32) * np.float32(scale / np.sqrt(d))).astype(np.float32)
    if dtype == "bf16":
        h, w = f32_to_bf16_bits(h), f32_to_bf16_bits(w)
    return h, w


def device_lm_head_inputs(rows: int, d: int, V: int, seed: int, device, scale: float = 2.0):
    """Device-resident ``(hidden[rows, d] bf16, weight[V, d] bf16)`` with the distributions of ``lm_head_inputs``."""
    import torch

    g = torch.Generator(device=device)
    g.manual_seed(int(seed) * 1_000_003 + 0x11E)
    h = torch.randn((rows, d), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    w = torch.empty((V, d), dtype=torch.bfloat16, device=device)
    step = max(1, (1 << 26) // d)
    for v0 in range(0, V, step):
        v1 = min(V, v0 + step)
        w[v0:v1] = (torch.randn((v1 - v0, d), generator=g, device=device, dtype=torch.float32)
                    * float(scale / np.sqrt(d))).to(torch.bfloat16)
    return h, w


def device_selector_tables(V: int, R: int, B: int, L: int, seed: int, device):
    """Device-resident stand-ins for the selector's tables: ``(phi[V,R] bf16, psi[V,R] bf16, gate[B,L,R] fp32,
    anchor_tokens[B] i32)``, same distributions as ``selector_tables``, drawn with a seeded torch generator."""
    import torch

    g = torch.Generator(device=device)
    g.manual_seed(int(seed) * 1_000_003 + 0x5E1)
    phi = torch.randn((V, R), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    psi = torch.randn((V, R), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    gate = torch.randn((B, L, R), generator=g, device=device, dtype=torch.float32) / float(np.sqrt(R))
    anchor = torch.randint(0, V, (B,), generator=g, device=device, dtype=torch.int32)
    return phi, psi, gate.contiguous(), anchor


def boost_children_on_device(z, token_ids, parents, n_nodes, boost: float) -> None:
    """Make device-resident target logits agree with a tree: in the row of every parent slot, the logit of
    each child's token is raised by ``boost`` (in place, rounded to the tensor's dtype).  With boost near
    log(V) a child is then picked with a probability of order one, so acceptance lengths are non-trivial.
    """
    import torch

    B, N = token_ids.shape
    slot = torch.arange(N, device=z.device)[None, :].expand(B, N)
    live = (slot >= 1) & (slot < n_nodes[:, None].to(z.device))
    b = torch.arange(B, device=z.device)[:, None].expand(B, N)[live]
    par = parents.to(z.device)[live].long()
    tok = token_ids.to(z.device)[live].long()
    cur = z[b, par, tok].float() + float(boost)
    z[b, par, tok] = cur.to(z.dtype)


def to_host_bits(t) -> np.ndarray:
    """Host copy of a torch tensor in this module's host representation."""
    import torch

    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def to_device(a: np.ndarray, dtype: str, device):
    """Upload a host tensor of this module to ``device`` as bf16 / fp32 / as-is."""
    import torch

    if dtype == "bf16" and a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(a).to(device)
