"""The per-rank partial of a vocabulary-parallel step a1 as include/ubt.h documents it, packed and unpacked with
numpy (test helper): four arrays, each starting on a 256-byte boundary: float32[rows,2] (max, sum of exp
relative to it), float32[rows,k] values best first, int32[rows,k] token ids of the whole vocabulary,
int32[rows] counts."""
import numpy as np


def _a256(n: int) -> int:
    return (n + 255) // 256 * 256


def offsets(rows: int, k: int):
    o_ms = 0
    o_val = o_ms + _a256(rows * 2 * 4)
    o_idx = o_val + _a256(rows * k * 4)
    o_cnt = o_idx + _a256(rows * k * 4)
    total = o_cnt + _a256(rows * 4)
    return o_ms, o_val, o_idx, o_cnt, total


def pack(ms: np.ndarray, val: np.ndarray, idx: np.ndarray, cnt: np.ndarray) -> np.ndarray:
    rows, k = val.shape
    o_ms, o_val, o_idx, o_cnt, total = offsets(rows, k)
    buf = np.zeros(total, np.uint8)
    buf[o_ms:o_ms + rows * 8] = np.ascontiguousarray(ms, np.float32).view(np.uint8).ravel()
    buf[o_val:o_val + rows * k * 4] = np.ascontiguousarray(val, np.float32).view(np.uint8).ravel()
    buf[o_idx:o_idx + rows * k * 4] = np.ascontiguousarray(idx, np.int32).view(np.uint8).ravel()
    buf[o_cnt:o_cnt + rows * 4] = np.ascontiguousarray(cnt, np.int32).view(np.uint8).ravel()
    return buf


def unpack(buf: np.ndarray, rows: int, k: int):
    o_ms, o_val, o_idx, o_cnt, total = offsets(rows, k)
    buf = np.ascontiguousarray(buf).view(np.uint8).ravel()
    assert buf.size >= total
    ms = buf[o_ms:o_ms + rows * 8].view(np.float32).reshape(rows, 2)
    val = buf[o_val:o_val + rows * k * 4].view(np.float32).reshape(rows, k)
    idx = buf[o_idx:o_idx + rows * k * 4].view(np.int32).reshape(rows, k)
    cnt = buf[o_cnt:o_cnt + rows * 4].view(np.int32).reshape(rows)
    return ms, val, idx, cnt


def merge(gathered: np.ndarray, shards: int, rows: int, k: int):
    """What ubt_topk_merge_shards computes, in double: (cand_ids[rows,k], cand_lp[rows,k])."""
    total = offsets(rows, k)[4]
    parts = [unpack(gathered[r * total:(r + 1) * total], rows, k) for r in range(shards)]
    ids = np.full((rows, k), -1, np.int32)
    lp = np.full((rows, k), -np.inf)
    for row in range(rows):
        m = max(float(p[0][row, 0]) for p in parts)
        s = sum(float(p[0][row, 1]) * np.exp(float(p[0][row, 0]) - m) for p in parts)
        lse = m + np.log(s)
        ent = [(-float(p[1][row, i]), int(p[2][row, i])) for p in parts for i in range(max(int(p[3][row]), 0))]
        ent.sort()
        for r, (nv, t) in enumerate(ent[:k]):
            ids[row, r] = t
            lp[row, r] = -nv - lse
    return ids, lp
