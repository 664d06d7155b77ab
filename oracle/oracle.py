"""CPU oracle for dynamic block-sparse attention.  TEST INFRASTRUCTURE ONLY.

Only ``tests/``, ``__graft_entry__.smoke()`` and ``bench.py``'s CPU-baseline leg
may import this package; the product (CUDA) path never does, and nothing here
imports the product package.  Everything is a plain restatement of what the
paper defines:

* ``attention_blocks`` / ``attention_full`` -- masked attention, Eq. 1 of
  Section 2.1, in fp64 (C, OpenMP), by expanding the block mask to token pairs.
* ``attention_bruteforce`` -- the same definition through an explicit N x N
  boolean matrix in numpy (tiny inputs only); pins the C routine.
* ``mask_stats`` -- active-block density and active-block-run coverage
  (Section 5.1), plus the row-nnz skew this build adds as a regime feature.
* ``active_runs`` -- maximal runs of consecutive active KV blocks (Section 4.3).
* ``block_csr`` -- block-CSR of a mask (Section 4.2, Section 5.2).
* ``coverage_counts`` -- how often each token-pair cell is covered by a list of
  physical tiles with membership bits; a plan preserves E(M) iff the count is
  1 on active cells and 0 elsewhere (Section 2.2 / 4.2).
* ``refine_columns`` -- KV-side refinement of a block-CSR column (Section 4.2).
* ``merge_partials`` -- Split-K merge of partial (O, LSE) states (Section 4.3).
* ``compile_table`` / ``select_plan`` -- Algorithm 1 and Algorithm 2.
* ``tile_flops`` / ``tile_kv_bytes`` / ``active_pairs`` -- the simplified bf16
  accounting of Section 2.3.

Parity pins: every function above is pinned by tests/test_oracle_pins.py to
something other than itself (textbook dense softmax, closed forms, the paper's
printed examples, brute force, invariants).  The numerical values of O have no
printed worked example in the paper; beyond those pins parity is oracle-only.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
from typing import Dict, Iterable, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libbsa_oracle.so")
_SRC_PATH = os.path.join(_HERE, "bsa_oracle.c")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc -O3 -march=native -fopenmp)."""
    if (not force) and os.path.exists(_LIB_PATH) and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(_SRC_PATH):
        return _LIB_PATH
    tmp = _LIB_PATH + f".{os.getpid()}.tmp"
    cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fno-fast-math", "-shared", "-fPIC", "-o", tmp, _SRC_PATH, "-lm"]
    subprocess.check_call(cmd)
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        # -march=native code must be built on the machine that runs it
        marker = _LIB_PATH + ".host"
        host = open("/proc/cpuinfo").read().split("model name")[1].split("\n")[0] if os.path.exists("/proc/cpuinfo") else ""
        stale = (not os.path.exists(marker)) or open(marker).read() != host
        build(force=stale)
        with open(marker, "w") as f:
            f.write(host)
        lib = ctypes.CDLL(_LIB_PATH)
        lib.bsa_oracle_blocks.restype = ctypes.c_int
        lib.bsa_oracle_blocks.argtypes = [
            ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int64,
            ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        lib.bsa_oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().bsa_oracle_num_threads())


def cdiv(a: int, b: int) -> int:
    return -(-a // b)


# --------------------------------------------------------------------------
# Eq. 1: masked attention
# --------------------------------------------------------------------------
def attention_blocks(mask: np.ndarray, B_Q: int, B_KV: int, N: int, d: int,
                     Qb: np.ndarray, Kb: np.ndarray, Vb: np.ndarray,
                     sel: Sequence[Tuple[int, int]], row_step: int = 1, N_kv: Optional[int] = None,
                     dtype: str = "bf16"):
    """Masked attention (Eq. 1) on selected (head, query-block) pairs.

    ``Qb`` is ``[H, N, d]`` and ``Kb/Vb`` are ``[H, N_kv, d]`` uint16 bf16 bit patterns (Section 2.1: N_q query
    and N_kv key tokens; ``N_kv`` defaults to ``N``), or IEEE half bit patterns with ``dtype="fp16"``.  Returns
    ``(O [n_sel, B_Q, d] float64, LSE [n_sel, B_Q] float64, active_pairs)``;
    rows at or beyond N, and rows skipped by ``row_step``, are NaN.
    """
    lib = _load()
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    H, nQb, nKb = mask.shape
    N_kv = N if N_kv is None else N_kv
    assert nQb == cdiv(N, B_Q) and nKb == cdiv(N_kv, B_KV)
    for a, n_tok in ((Qb, N), (Kb, N_kv), (Vb, N_kv)):
        assert a.dtype == np.uint16 and a.shape == (H, n_tok, d) and a.flags.c_contiguous
    sel_h = np.ascontiguousarray([s[0] for s in sel], dtype=np.int32)
    sel_b = np.ascontiguousarray([s[1] for s in sel], dtype=np.int32)
    n = len(sel_h)
    O = np.full((n, B_Q, d), np.nan, dtype=np.float64)
    LSE = np.full((n, B_Q), np.nan, dtype=np.float64)
    pairs = ctypes.c_int64(0)
    assert dtype in ("bf16", "fp16")
    rc = lib.bsa_oracle_blocks(mask.ctypes.data, H, nQb, nKb, B_Q, B_KV, N, N_kv, d, int(dtype == "fp16"), Qb.ctypes.data, Kb.ctypes.data,
                               Vb.ctypes.data, n, sel_h.ctypes.data, sel_b.ctypes.data, row_step,
                               O.ctypes.data, LSE.ctypes.data, ctypes.byref(pairs))
    if rc != 0:
        raise MemoryError("oracle allocation failed")
    return O, LSE, int(pairs.value)


def attention_full(mask, B_Q, B_KV, N, d, Qb, Kb, Vb, N_kv=None, dtype="bf16"):
    """Eq. 1 on every row.  Returns ``O [H, N, d]`` and ``LSE [H, N]`` (float64)."""
    H, nQb, _ = mask.shape
    sel = [(h, i) for h in range(H) for i in range(nQb)]
    O, LSE, pairs = attention_blocks(mask, B_Q, B_KV, N, d, Qb, Kb, Vb, sel, N_kv=N_kv, dtype=dtype)
    O = O.reshape(H, nQb * B_Q, d)[:, :N]
    LSE = LSE.reshape(H, nQb * B_Q)[:, :N]
    return np.ascontiguousarray(O), np.ascontiguousarray(LSE), pairs


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def bits_to_f64(b: np.ndarray, dtype: str = "bf16") -> np.ndarray:
    """16-bit patterns to float64: bf16, or IEEE half through numpy's own float16."""
    return np.ascontiguousarray(b).view(np.float16).astype(np.float64) if dtype == "fp16" else bf16_bits_to_f64(b)


def expand_mask(mask_h: np.ndarray, B_Q: int, B_KV: int, N: int, N_kv=None) -> np.ndarray:
    """E(M) of one head as an explicit ``[N, N_kv]`` boolean matrix (Section 2.1)."""
    return np.repeat(np.repeat(mask_h != 0, B_Q, axis=0), B_KV, axis=1)[:N, :(N if N_kv is None else N_kv)]


def attention_bruteforce(mask, B_Q, B_KV, N, d, Qb, Kb, Vb, N_kv=None, dtype="bf16"):
    """Eq. 1 through an explicit token-pair matrix, one row at a time (tiny inputs)."""
    H = mask.shape[0]
    Q, K, V = (bits_to_f64(x, dtype) for x in (Qb, Kb, Vb))
    O = np.zeros((H, N, d))
    LSE = np.full((H, N), -np.inf)
    for h in range(H):
        E = expand_mask(mask[h], B_Q, B_KV, N, N_kv)
        for i in range(N):
            J = np.nonzero(E[i])[0]
            if J.size == 0:
                continue
            s = (K[h, J] @ Q[h, i]) / math.sqrt(d)
            m = s.max()
            p = np.exp(s - m)
            l = p.sum()
            O[h, i] = (p[:, None] * V[h, J]).sum(axis=0) / l
            LSE[h, i] = m + math.log(l)
    return O, LSE


# --------------------------------------------------------------------------
# Section 2.3 accounting
# --------------------------------------------------------------------------
def active_pairs(mask: np.ndarray, B_Q: int, B_KV: int, N: int, N_kv=None) -> int:
    """Number of in-range token pairs in E(M), all heads."""
    H, nQb, nKb = mask.shape
    rq = np.minimum(B_Q, N - np.arange(nQb) * B_Q).astype(np.int64)
    ck = np.minimum(B_KV, (N if N_kv is None else N_kv) - np.arange(nKb) * B_KV).astype(np.int64)
    return int(((mask != 0).astype(np.int64) * rq[None, :, None] * ck[None, None, :]).sum())


def tile_flops(d: int, T_Q: int, T_KV: int) -> int:
    """About 4 d T_Q T_KV flops per physical tile (QK^T plus PV)."""
    return 4 * d * T_Q * T_KV


def tile_kv_bytes(d: int, T_KV: int) -> int:
    """About 4 d T_KV bytes of K and V per tile in bf16."""
    return 4 * d * T_KV


# --------------------------------------------------------------------------
# Section 4.3 / 5.1: runs and scalar mask statistics
# --------------------------------------------------------------------------
def active_runs(cols: Iterable[int]) -> List[Tuple[int, int]]:
    """Maximal runs of consecutive active KV block indices of one query-block row."""
    runs: List[Tuple[int, int]] = []
    for c in sorted(set(int(x) for x in cols)):
        if runs and runs[-1][1] + 1 == c:
            runs[-1] = (runs[-1][0], c)
        else:
            runs.append((c, c))
    return runs


def mask_stats(mask: np.ndarray) -> Dict[str, float]:
    """density = active / all logical blocks; run coverage = fraction of active
    blocks in runs of length >= 2 (0 for an empty mask); skew = max row nnz over
    mean row nnz (0 for an empty mask).  Runs never cross rows or heads."""
    H, nQb, nKb = mask.shape
    nnz = 0
    in_runs = 0
    max_row = 0
    for h in range(H):
        for i in range(nQb):
            cols = np.nonzero(mask[h, i])[0]
            nnz += cols.size
            max_row = max(max_row, int(cols.size))
            for a, b in active_runs(cols):
                if b - a + 1 >= 2:
                    in_runs += b - a + 1
    total = H * nQb * nKb
    return {
        "nnz": nnz,
        "density": nnz / total if total else 0.0,
        "run_coverage": in_runs / nnz if nnz else 0.0,
        "max_row_nnz": max_row,
        "skew": max_row / (nnz / (H * nQb)) if nnz else 0.0,
        "blocks_in_runs": in_runs,
    }


def block_csr(mask: np.ndarray):
    """Per head: row offsets and sorted active KV column indices, heads concatenated.
    Returns ``(row_ptr int32 [H*nQb+1], col_idx int32 [nnz])``."""
    H, nQb, nKb = mask.shape
    counts = (mask != 0).sum(axis=2).reshape(-1)
    row_ptr = np.zeros(H * nQb + 1, dtype=np.int64)
    np.cumsum(counts, out=row_ptr[1:])
    col_idx = np.nonzero(mask.reshape(H * nQb, nKb))[1].astype(np.int32)
    return row_ptr.astype(np.int32), col_idx


def refine_columns(c: int, ratio: int) -> List[int]:
    """KV-side refinement: block column ``c`` names ``ratio`` finer tiles."""
    return [c * ratio + k for k in range(ratio)]


# --------------------------------------------------------------------------
# plan coverage: does a set of physical tiles preserve E(M)?
# --------------------------------------------------------------------------
def coverage_counts(H: int, N: int, B_Q: int, B_KV: int, T_Q: int, T_KV: int,
                    tiles: Dict[int, Tuple[np.ndarray, np.ndarray, np.ndarray]], N_kv=None) -> np.ndarray:
    """Count how many tiles cover each cell, honouring membership bits.

    A cell is ``min(B_Q,T_Q) x min(B_KV,T_KV)`` tokens; every block and every
    tile is a union of cells, so equality on cells is equality on token pairs.
    ``tiles[h] = (tile_row_ptr [nQt+1], tile_col [n], tile_member [n] uint64)``
    with tile_row_ptr relative to that head's arrays.  Membership bit
    ``a * sK + b`` (``sQ = max(1, T_Q // B_Q)``, ``sK = max(1, T_KV // B_KV)``,
    ``a < sQ``, ``b < sK``) says logical sub-block (a, b) of the tile is active;
    bits of sub-blocks that start at or beyond N (rows) or N_kv (columns, default N) must be clear.
    Returns int32 ``[H, nCq, nCk]``.
    """
    cq, ck = min(B_Q, T_Q), min(B_KV, T_KV)
    nCq, nCk = cdiv(N, cq), cdiv(N if N_kv is None else N_kv, ck)
    sQ, sK = max(1, T_Q // B_Q), max(1, T_KV // B_KV)
    cells_q, cells_k = T_Q // cq, T_KV // ck  # cells per tile edge
    cover = np.zeros((H, nCq, nCk), dtype=np.int32)
    for h, (rp, tc, tm) in tiles.items():
        nQt = len(rp) - 1
        for t in range(nQt):
            for idx in range(int(rp[t]), int(rp[t + 1])):
                c = int(tc[idx])
                mem = int(tm[idx])
                for a in range(cells_q):
                    for b in range(cells_k):
                        # which logical sub-block of the tile this cell belongs to
                        sa = a if sQ > 1 else 0
                        sb = b if sK > 1 else 0
                        if not (mem >> (sa * sK + sb)) & 1:
                            continue
                        gq, gk = t * cells_q + a, c * cells_k + b
                        if gq < nCq and gk < nCk:
                            cover[h, gq, gk] += 1
                        else:
                            raise AssertionError(f"tile ({h},{t},{c}) marks an out-of-range cell active")
    return cover


def expected_cell_cover(mask: np.ndarray, N: int, B_Q: int, B_KV: int, T_Q: int, T_KV: int, N_kv=None) -> np.ndarray:
    """E(M) at cell granularity: 1 on cells of active blocks, else 0."""
    cq, ck = min(B_Q, T_Q), min(B_KV, T_KV)
    nCq, nCk = cdiv(N, cq), cdiv(N if N_kv is None else N_kv, ck)
    e = np.repeat(np.repeat((mask != 0).astype(np.int32), B_Q // cq, axis=1), B_KV // ck, axis=2)
    return np.ascontiguousarray(e[:, :nCq, :nCk])


# --------------------------------------------------------------------------
# Split-K merge (Section 4.3): rescale partial states to a common maximum,
# merge, normalise.  With partials stored as (normalised O_p, LSE_p) this is
# LSE = logsumexp_p LSE_p and O = sum_p exp(LSE_p - LSE) O_p.
# --------------------------------------------------------------------------
def merge_partials(Os: Sequence[np.ndarray], LSEs: Sequence[np.ndarray]):
    Os = [np.asarray(o, dtype=np.float64) for o in Os]
    LSEs = [np.asarray(l, dtype=np.float64) for l in LSEs]
    m = np.maximum.reduce(LSEs)
    m_safe = np.where(np.isfinite(m), m, 0.0)
    w = [np.exp(l - m_safe) for l in LSEs]  # exp(-inf) = 0 for empty partitions
    tot = np.add.reduce(w)
    with np.errstate(divide="ignore", invalid="ignore"):
        O = np.add.reduce([wi[..., None] * o for wi, o in zip(w, Os)]) / np.where(tot > 0, tot, 1.0)[..., None]
        LSE = np.where(tot > 0, m_safe + np.log(np.where(tot > 0, tot, 1.0)), -np.inf)
    return O, LSE


# --------------------------------------------------------------------------
# Algorithm 1 (offline table compilation) and Algorithm 2 (online selection)
# --------------------------------------------------------------------------
def compile_table(cases, latencies, base_plan, bucket_of):
    """Algorithm 1, regimes-and-rankings half.

    cases     : list of (case_id, request_key)
    latencies : dict (case_id, plan_id) -> validated median latency (absent = not valid)
    base_plan : dict request_key -> plan_id
    bucket_of : callable case_id -> hashable bucket
    Returns dict (request_key, bucket) -> [ranked plan ids..., base plan].
    """
    table = {}
    keys = sorted(set(k for _, k in cases), key=repr)
    for k in keys:
        Mk = [c for c, kk in cases if kk == k]
        buckets = {}
        for c in Mk:
            buckets.setdefault(bucket_of(c), []).append(c)
        for b, members in buckets.items():
            plans = set(p for (c, p) in latencies if c in members)
            Cb = [p for p in plans if all((c, p) in latencies for c in members)]
            if not Cb:
                continue
            gm = {p: math.exp(sum(math.log(latencies[(c, p)]) for c in members) / len(members)) for p in Cb}
            Cb.sort(key=lambda p: (gm[p], p))
            table[(k, b)] = Cb + [base_plan[k]]
    return table


def select_plan(table, base_plan, key, bucket, eligible):
    """Algorithm 2: ranked list of the regime (base plan alone on a miss); first
    eligible plan wins; ``None`` stands for no-eligible-plan."""
    ranked = table.get((key, bucket))
    if ranked is None:
        ranked = [base_plan[key]] if key in base_plan else []
    for p in ranked:
        if eligible(p):
            return p
    return None
