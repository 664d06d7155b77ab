"""Pins for the CPU oracle: each check compares it with something other than
itself -- a textbook routine, a closed form, a value the paper prints, brute
force on tiny inputs, or an invariant of masked attention (Eq. 1, Section 2.1).
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_25869_b200 import inputs as I

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _bits(x: np.ndarray) -> np.ndarray:
    """float array -> bf16 bit patterns (round to nearest even)."""
    return I.bf16_bits(torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16))


def _small(seed, H, N, d):
    q, k, v = I.make_qkv(seed, H, N, d)
    return I.bf16_bits(q), I.bf16_bits(k), I.bf16_bits(v), (q, k, v)


# ---------------------------------------------------------------- Eq. 1
def test_all_ones_mask_is_dense_softmax_attention():
    H, N, d, B = 2, 192, 64, 64
    Qb, Kb, Vb, (q, k, v) = _small(11, H, N, d)
    M = np.ones((H, N // B, N // B), dtype=np.uint8)
    O, LSE, pairs = oracle.attention_full(M, B, B, N, d, Qb, Kb, Vb)
    q64, k64, v64 = (t.to(torch.float64) for t in (q, k, v))
    s = q64 @ k64.transpose(1, 2) / math.sqrt(d)
    ref_O = torch.softmax(s, dim=-1) @ v64
    ref_L = torch.logsumexp(s, dim=-1)
    assert pairs == H * N * N
    np.testing.assert_allclose(O, ref_O.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(LSE, ref_L.numpy(), rtol=0, atol=1e-12)


def test_dense_softmax_with_more_keys_than_queries_and_fewer():
    """Section 2.1: Q is N_q x d, K and V are N_kv x d.  With every block active the result is the textbook
    softmax(Q K^T / sqrt(d)) V of the rectangular score matrix (ragged last blocks on both sides)."""
    H, d, B_Q, B_KV = 2, 32, 32, 64
    for N_q, N_kv in ((70, 200), (200, 70)):
        q, _, _ = I.make_qkv(21, H, N_q, d)
        _, k, v = I.make_qkv(22, H, N_kv, d)
        M = np.ones((H, I.cdiv(N_q, B_Q), I.cdiv(N_kv, B_KV)), dtype=np.uint8)
        O, LSE, pairs = oracle.attention_full(M, B_Q, B_KV, N_q, d, I.bf16_bits(q), I.bf16_bits(k), I.bf16_bits(v),
                                              N_kv=N_kv)
        q64, k64, v64 = (t.to(torch.float64) for t in (q, k, v))
        s = q64 @ k64.transpose(1, 2) / math.sqrt(d)
        assert pairs == H * N_q * N_kv == oracle.active_pairs(M, B_Q, B_KV, N_q, N_kv)
        assert O.shape == (H, N_q, d)
        np.testing.assert_allclose(O, (torch.softmax(s, dim=-1) @ v64).numpy(), rtol=0, atol=1e-12)
        np.testing.assert_allclose(LSE, torch.logsumexp(s, dim=-1).numpy(), rtol=0, atol=1e-12)


@pytest.mark.parametrize("B_Q,B_KV,N_q,N_kv", [(16, 32, 50, 130), (64, 16, 130, 40)])
def test_bruteforce_token_pair_matrix_rectangular(B_Q, B_KV, N_q, N_kv):
    H, d = 2, 16
    q, _, _ = I.make_qkv(31, H, N_q, d)
    _, k, v = I.make_qkv(32, H, N_kv, d)
    Qb, Kb, Vb = I.bf16_bits(q), I.bf16_bits(k), I.bf16_bits(v)
    M = I.random_mask(9, H, I.cdiv(N_q, B_Q), I.cdiv(N_kv, B_KV), 0.4, empty_rows=0.2)
    O, LSE, pairs = oracle.attention_full(M, B_Q, B_KV, N_q, d, Qb, Kb, Vb, N_kv=N_kv)
    bO, bL = oracle.attention_bruteforce(M, B_Q, B_KV, N_q, d, Qb, Kb, Vb, N_kv=N_kv)
    np.testing.assert_allclose(O, bO, rtol=0, atol=1e-13)
    assert np.array_equal(np.isneginf(LSE), np.isneginf(bL))
    fin = np.isfinite(bL)
    np.testing.assert_allclose(LSE[fin], bL[fin], rtol=0, atol=1e-13)
    E = sum(int(oracle.expand_mask(M[h], B_Q, B_KV, N_q, N_kv).sum()) for h in range(H))
    assert pairs == E == oracle.active_pairs(M, B_Q, B_KV, N_q, N_kv)


def test_half_precision_inputs_dense_softmax_and_bruteforce():
    """Tensor type as a request property (Section 4.4): IEEE half inputs, widened exactly.  Dense mask against
    torch's softmax on torch's own half -> double conversion (normal, subnormal and zero values included), and a
    sparse mask against the brute force, which converts through numpy's float16."""
    H, N, d, B = 2, 96, 32, 32
    q, k, v = I.make_qkv(51, H, N, d, dtype="fp16")
    assert q.dtype == torch.float16
    k[0, 0, :4] = torch.tensor([6e-8, -3e-6, 0.0, 65504.0 / 4096], dtype=torch.float16)  # subnormals, zero
    q[0, 1, :4] = torch.tensor([5.96e-8, 1e-7, -0.0, 2.0], dtype=torch.float16)
    Qb, Kb, Vb = I.bf16_bits(q), I.bf16_bits(k), I.bf16_bits(v)
    M = np.ones((H, N // B, N // B), dtype=np.uint8)
    O, LSE, _ = oracle.attention_full(M, B, B, N, d, Qb, Kb, Vb, dtype="fp16")
    q64, k64, v64 = (t.to(torch.float64) for t in (q, k, v))
    s = q64 @ k64.transpose(1, 2) / math.sqrt(d)
    np.testing.assert_allclose(O, (torch.softmax(s, dim=-1) @ v64).numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(LSE, torch.logsumexp(s, dim=-1).numpy(), rtol=0, atol=1e-12)
    # the same bits read as bf16 are other numbers: the flag matters
    O_b, _, _ = oracle.attention_full(M, B, B, N, d, Qb, Kb, Vb)
    assert np.abs(O_b - O).max() > 1e-3
    Ms = I.random_mask(3, H, N // B, N // B, 0.5, empty_rows=0.3)
    O, LSE, _ = oracle.attention_full(Ms, B, B, N, d, Qb, Kb, Vb, dtype="fp16")
    bO, bL = oracle.attention_bruteforce(Ms, B, B, N, d, Qb, Kb, Vb, dtype="fp16")
    np.testing.assert_allclose(O, bO, rtol=0, atol=1e-13)
    fin = np.isfinite(bL)
    assert np.array_equal(np.isfinite(LSE), fin)
    np.testing.assert_allclose(LSE[fin], bL[fin], rtol=0, atol=1e-13)


def test_hand_computed_two_keys():
    # d = 4, one query q = (2,0,0,0), keys k0 = (2,0,0,0), k1 = (-2,0,0,0): scores 4/2 = 2 and -2.
    N, d = 2, 4
    Q = np.zeros((1, N, d)); K = np.zeros((1, N, d)); V = np.zeros((1, N, d))
    Q[0, 0, 0] = 2.0
    Q[0, 1, 0] = 0.0
    K[0, 0, 0] = 2.0
    K[0, 1, 0] = -2.0
    V[0, 0] = [1, 0, 0, 8]
    V[0, 1] = [3, 0, 0, -8]
    M = np.ones((1, 1, 1), dtype=np.uint8)
    O, LSE, _ = oracle.attention_full(M, 2, 2, N, d, _bits(Q), _bits(K), _bits(V))
    e2, em2 = math.exp(2.0), math.exp(-2.0)
    assert LSE[0, 0] == pytest.approx(math.log(e2 + em2), abs=1e-14)
    assert O[0, 0, 0] == pytest.approx((e2 * 1 + em2 * 3) / (e2 + em2), abs=1e-14)
    assert O[0, 0, 3] == pytest.approx((e2 * 8 - em2 * 8) / (e2 + em2), abs=1e-14)
    # second query is all zero: uniform average, LSE = ln 2
    assert LSE[0, 1] == pytest.approx(math.log(2.0), abs=1e-14)
    np.testing.assert_allclose(O[0, 1], [2, 0, 0, 0], atol=1e-14)


@pytest.mark.parametrize("B_Q,B_KV,N", [(16, 16, 64), (16, 64, 128), (64, 16, 128), (32, 64, 200), (64, 32, 130)])
def test_bruteforce_token_pair_matrix(B_Q, B_KV, N):
    H, d = 2, 16
    Qb, Kb, Vb, _ = _small(5 + N, H, N, d)
    M = I.random_mask(7, H, I.cdiv(N, B_Q), I.cdiv(N, B_KV), 0.4, empty_rows=0.2)
    O, LSE, pairs = oracle.attention_full(M, B_Q, B_KV, N, d, Qb, Kb, Vb)
    bO, bL = oracle.attention_bruteforce(M, B_Q, B_KV, N, d, Qb, Kb, Vb)
    np.testing.assert_allclose(O, bO, rtol=0, atol=1e-13)
    assert np.array_equal(np.isneginf(LSE), np.isneginf(bL))
    fin = np.isfinite(bL)
    np.testing.assert_allclose(LSE[fin], bL[fin], rtol=0, atol=1e-13)
    E = sum(int(oracle.expand_mask(M[h], B_Q, B_KV, N).sum()) for h in range(H))
    assert pairs == E == oracle.active_pairs(M, B_Q, B_KV, N)


@pytest.mark.parametrize("B_Q,B_KV,N", [(32, 16, 96), (16, 64, 150)])
def test_closed_forms_zero_keys_and_constant_values(B_Q, B_KV, N):
    H, d = 2, 8
    Qb, Kb, Vb, (q, k, v) = _small(3, H, N, d)
    M = I.random_mask(9, H, I.cdiv(N, B_Q), I.cdiv(N, B_KV), 0.5, empty_rows=0.25)
    # K = 0: every reachable score is 0, so LSE = ln #J and O = mean of reachable V
    O, LSE, _ = oracle.attention_full(M, B_Q, B_KV, N, d, Qb, np.zeros_like(Kb), Vb)
    V64 = oracle.bf16_bits_to_f64(Vb)
    for h in range(H):
        E = oracle.expand_mask(M[h], B_Q, B_KV, N)
        cnt = E.sum(axis=1)
        for i in range(N):
            if cnt[i] == 0:
                assert LSE[h, i] == -np.inf and not O[h, i].any()
            else:
                assert LSE[h, i] == pytest.approx(math.log(cnt[i]), abs=1e-13)
                np.testing.assert_allclose(O[h, i], V64[h, E[i]].mean(axis=0), atol=1e-13)
    # V = const c: O = c on non-empty rows
    c = 0.75
    Vc = _bits(np.full((H, N, d), c))
    O2, L2, _ = oracle.attention_full(M, B_Q, B_KV, N, d, Qb, Kb, Vc)
    nonempty = np.isfinite(L2)
    np.testing.assert_allclose(O2[nonempty], c, atol=1e-13)
    assert not O2[~nonempty].any()
    # every output lies inside the per-dimension range of the values
    O3, L3, _ = oracle.attention_full(M, B_Q, B_KV, N, d, Qb, Kb, Vb)
    for h in range(H):
        E = oracle.expand_mask(M[h], B_Q, B_KV, N)
        for i in np.nonzero(E.any(axis=1))[0]:
            vv = V64[h, E[i]]
            assert (O3[h, i] <= vv.max(axis=0) + 1e-12).all() and (O3[h, i] >= vv.min(axis=0) - 1e-12).all()


def test_rows_with_no_active_block():
    H, N, d, B = 1, 128, 16, 32
    Qb, Kb, Vb, _ = _small(2, H, N, d)
    M = np.zeros((H, 4, 4), dtype=np.uint8)
    M[0, 1, 2] = 1
    O, LSE, pairs = oracle.attention_full(M, B, B, N, d, Qb, Kb, Vb)
    assert pairs == 32 * 32
    for blk in (0, 2, 3):
        assert not O[0, blk * B:(blk + 1) * B].any()
        assert np.isneginf(LSE[0, blk * B:(blk + 1) * B]).all()
    assert np.isfinite(LSE[0, B:2 * B]).all()


def test_permuting_keys_inside_a_block_changes_nothing():
    H, N, d, B_Q, B_KV = 1, 128, 16, 16, 32
    Qb, Kb, Vb, _ = _small(4, H, N, d)
    M = I.random_mask(1, H, N // B_Q, N // B_KV, 0.5, diag=True)
    O, LSE, _ = oracle.attention_full(M, B_Q, B_KV, N, d, Qb, Kb, Vb)
    perm = np.arange(N)
    rng = np.random.default_rng(0)
    for b in range(N // B_KV):
        perm[b * B_KV:(b + 1) * B_KV] = b * B_KV + rng.permutation(B_KV)
    O2, L2, _ = oracle.attention_full(M, B_Q, B_KV, N, d, Qb, np.ascontiguousarray(Kb[:, perm]),
                                      np.ascontiguousarray(Vb[:, perm]))
    np.testing.assert_allclose(O2, O, atol=1e-13)
    np.testing.assert_allclose(L2, LSE, atol=1e-13)
    # permuting ACROSS blocks must change a sparse result (guards against a no-op test)
    perm2 = np.roll(np.arange(N), B_KV)
    O3, _, _ = oracle.attention_full(M, B_Q, B_KV, N, d, Qb, np.ascontiguousarray(Kb[:, perm2]),
                                     np.ascontiguousarray(Vb[:, perm2]))
    assert np.abs(O3 - O).max() > 1e-3


def test_unreachable_keys_do_not_matter():
    H, N, d, B_Q, B_KV = 1, 96, 8, 32, 16
    Qb, Kb, Vb, _ = _small(6, H, N, d)
    M = np.zeros((H, 3, 6), dtype=np.uint8)
    M[0, 0, [0, 3]] = 1
    M[0, 1, [1]] = 1
    M[0, 2, [4, 5]] = 1
    O, LSE, _ = oracle.attention_full(M, B_Q, B_KV, N, d, Qb, Kb, Vb)
    K2, V2 = Kb.copy(), Vb.copy()
    K2[0, 2 * B_KV:3 * B_KV] = _bits(np.full((B_KV, d), 7.0))  # KV block 2 is reached by no row
    V2[0, 2 * B_KV:3 * B_KV] = _bits(np.full((B_KV, d), -9.0))
    O2, L2, _ = oracle.attention_full(M, B_Q, B_KV, N, d, Qb, K2, V2)
    assert np.array_equal(O, O2) and np.array_equal(LSE, L2)
    # block 1 is reached only by row-block 1: other rows stay bit-identical, those rows change
    K3 = Kb.copy()
    K3[0, B_KV:2 * B_KV] = _bits(np.full((B_KV, d), 1.5))
    O3, L3, _ = oracle.attention_full(M, B_Q, B_KV, N, d, Qb, K3, Vb)
    assert np.array_equal(O3[0, :32], O[0, :32]) and np.array_equal(O3[0, 64:], O[0, 64:])
    assert not np.array_equal(L3[0, 32:64], LSE[0, 32:64])


# ---------------------------------------------------------------- Split-K merge
def test_merge_of_disjoint_masks_equals_union():
    H, N, d, B_Q, B_KV = 2, 128, 16, 32, 16
    Qb, Kb, Vb, _ = _small(8, H, N, d)
    M = I.random_mask(3, H, N // B_Q, N // B_KV, 0.5, empty_rows=0.2)
    split = I.random_mask(4, H, N // B_Q, N // B_KV, 0.5)
    M1, M2 = M * split, M * (1 - split)
    M3 = np.zeros_like(M)  # an empty partition has weight 0
    parts = [oracle.attention_full(m, B_Q, B_KV, N, d, Qb, Kb, Vb)[:2] for m in (M1, M2, M3)]
    O, LSE = oracle.merge_partials([p[0] for p in parts], [p[1] for p in parts])
    rO, rL, _ = oracle.attention_full(M, B_Q, B_KV, N, d, Qb, Kb, Vb)
    np.testing.assert_allclose(O, rO, atol=1e-12)
    assert np.array_equal(np.isneginf(LSE), np.isneginf(rL))
    fin = np.isfinite(rL)
    np.testing.assert_allclose(LSE[fin], rL[fin], atol=1e-12)


# ---------------------------------------------------------------- runs / stats (paper's printed example)
def test_runs_example_from_the_paper():
    cols, runs = None, []
    for line in open(os.path.join(GOLD, "runs_example.txt")):
        t = line.split()
        if not t or t[0].startswith("#"):
            continue
        if t[0] == "cols":
            cols = [int(x) for x in t[1:]]
        elif t[0] == "run":
            runs.append((int(t[1]), int(t[2])))
    assert oracle.active_runs(cols) == runs
    M = np.zeros((1, 1, 12), dtype=np.uint8)
    M[0, 0, cols] = 1
    st = oracle.mask_stats(M)
    assert st["run_coverage"] == pytest.approx(3 / 4)
    assert st["density"] == pytest.approx(4 / 12)


def test_stats_empty_and_full_and_rows_do_not_join():
    assert oracle.mask_stats(np.zeros((2, 3, 5), np.uint8)) == {
        "nnz": 0, "density": 0.0, "run_coverage": 0.0, "max_row_nnz": 0, "skew": 0.0, "blocks_in_runs": 0}
    st = oracle.mask_stats(np.ones((2, 3, 5), np.uint8))
    assert st["density"] == 1.0 and st["run_coverage"] == 1.0 and st["skew"] == 1.0
    # last block of row 0 and first block of row 1 are adjacent in memory but not a run
    M = np.zeros((1, 2, 4), np.uint8)
    M[0, 0, 3] = 1
    M[0, 1, 0] = 1
    st = oracle.mask_stats(M)
    assert st["run_coverage"] == 0.0 and st["skew"] == 1.0
    M[0, 1, 1] = 1
    st = oracle.mask_stats(M)
    assert st["run_coverage"] == pytest.approx(2 / 3) and st["skew"] == pytest.approx(2 / 1.5)


def test_block_csr_roundtrip():
    M = I.random_mask(5, 3, 7, 9, 0.3, empty_rows=0.3)
    rp, ci = oracle.block_csr(M)
    back = np.zeros_like(M).reshape(-1, 9)
    for r in range(3 * 7):
        cols = ci[rp[r]:rp[r + 1]]
        assert (np.diff(cols) > 0).all()
        back[r, cols] = 1
    assert np.array_equal(back.reshape(M.shape), M)


# ---------------------------------------------------------------- refinement / coverage (paper's printed example)
def test_refined_example_from_the_paper():
    g = {}
    for line in open(os.path.join(GOLD, "refine_example.txt")):
        t = line.split()
        if t and not t[0].startswith("#"):
            g[t[0]] = int(t[1])
    for c in (0, 3, 7):
        assert oracle.refine_columns(c, g["kv_ratio"]) == [2 * c, 2 * c + 1]
    # one active 128x128 block at (1, 3) of a 4x4 mask -> four 64x64 tiles cover it exactly
    N = 512
    M = np.zeros((1, 4, 4), np.uint8)
    M[0, 1, 3] = 1
    rows = {1 * g["q_ratio"] + a: oracle.refine_columns(3, g["kv_ratio"]) for a in range(g["q_ratio"])}
    nQt = N // g["T_Q"]
    rp = np.zeros(nQt + 1, np.int64)
    tc = []
    for t in range(nQt):
        tc += rows.get(t, [])
        rp[t + 1] = len(tc)
    assert len(tc) == g["tiles_per_block"]
    tiles = {0: (rp, np.array(tc), np.ones(len(tc), np.uint64))}
    cover = oracle.coverage_counts(1, N, g["B_Q"], g["B_KV"], g["T_Q"], g["T_KV"], tiles)
    assert np.array_equal(cover, oracle.expected_cell_cover(M, N, g["B_Q"], g["B_KV"], g["T_Q"], g["T_KV"]))
    # dropping one of the four tiles, or doubling one, must be caught
    bad = {0: (np.minimum(rp, 3), np.array(tc[:3]), np.ones(3, np.uint64))}
    assert not np.array_equal(oracle.coverage_counts(1, N, 128, 128, 64, 64, bad),
                              oracle.expected_cell_cover(M, N, 128, 128, 64, 64))


def test_coverage_counts_coarsened_membership_bits():
    # B = (16, 32), T = (64, 64): 4 x 2 sub-blocks per tile, bit a*2+b
    N, B_Q, B_KV, T_Q, T_KV = 128, 16, 32, 64, 64
    M = np.zeros((1, 8, 4), np.uint8)
    M[0, 0, 0] = 1      # tile (0,0) sub (0,0)
    M[0, 3, 1] = 1      # tile (0,0) sub (3,1)
    M[0, 5, 2] = 1      # tile (1,1) sub (1,0)
    tiles = {0: (np.array([0, 1, 2]), np.array([0, 1]), np.array([(1 << 0) | (1 << 7), 1 << 2], np.uint64))}
    cover = oracle.coverage_counts(1, N, B_Q, B_KV, T_Q, T_KV, tiles)
    assert np.array_equal(cover, oracle.expected_cell_cover(M, N, B_Q, B_KV, T_Q, T_KV))
    wrong = {0: (np.array([0, 1, 2]), np.array([0, 1]), np.array([(1 << 0) | (1 << 6), 1 << 2], np.uint64))}
    assert not np.array_equal(oracle.coverage_counts(1, N, B_Q, B_KV, T_Q, T_KV, wrong),
                              oracle.expected_cell_cover(M, N, B_Q, B_KV, T_Q, T_KV))


def test_tile_accounting_from_the_paper():
    for line in open(os.path.join(GOLD, "accounting.txt")):
        t = line.split()
        if not t or t[0].startswith("#"):
            continue
        d, tq, tk, fl, by = (int(x) for x in t)
        assert oracle.tile_flops(d, tq, tk) == fl
        assert oracle.tile_kv_bytes(d, tk) == by
        assert fl / by == tq  # ratio approaches T_Q flop per byte with Q resident


# ---------------------------------------------------------------- Algorithm 1 / Algorithm 2
def test_table_compilation_and_selection_hand_computed():
    key = ("B200", (128, 128), ("bf16", 128))
    cases = [("c1", key), ("c2", key), ("c3", key), ("d1", ("B200", (64, 64), ("bf16", 64)))]
    lat = {
        ("c1", 0): 4.0, ("c2", 0): 1.0,              # plan 0: geo-mean 2.0 on bucket {c1, c2}
        ("c1", 1): 2.0, ("c2", 1): 2.0,              # plan 1: geo-mean 2.0 -> exact tie, lower id first
        ("c1", 2): 1.0,                                # plan 2: invalid on c2 -> not ranked in that bucket
        ("c3", 2): 1.0, ("c3", 0): 3.0, ("c3", 1): 2.0,
        ("d1", 5): 1.0,
    }
    base = {key: 9, ("B200", (64, 64), ("bf16", 64)): 5}
    bucket = {"c1": "lo", "c2": "lo", "c3": "hi", "d1": "lo"}.get
    table = oracle.compile_table(cases, lat, base, bucket)
    assert table[(key, "lo")] == [0, 1, 9]
    assert table[(key, "hi")] == [2, 1, 0, 9]
    assert table[(("B200", (64, 64), ("bf16", 64)), "lo")] == [5, 5]
    # Algorithm 2: first eligible in rank order; miss -> base plan only; nothing eligible -> None
    assert oracle.select_plan(table, base, key, "hi", lambda p: True) == 2
    assert oracle.select_plan(table, base, key, "hi", lambda p: p != 2) == 1
    assert oracle.select_plan(table, base, key, "mid", lambda p: True) == 9
    assert oracle.select_plan(table, base, key, "mid", lambda p: p != 9) is None
    assert oracle.select_plan(table, base, key, "lo", lambda p: False) is None
    assert oracle.select_plan(table, base, ("H100", (1, 1), ()), "lo", lambda p: True) is None


# ---------------------------------------------------------------- sampled evaluation equals full evaluation
def test_block_sample_matches_full_and_row_step():
    r = I.config_tiny()
    q, k, v = r.qkv()
    Qb, Kb, Vb = (I.bf16_bits(t) for t in (q, k, v))
    O, LSE, _ = oracle.attention_full(r.mask, r.B_Q, r.B_KV, r.N, r.d, Qb, Kb, Vb)
    sel = [(1, 5), (0, 31), (1, 0)]
    Os, Ls, _ = oracle.attention_blocks(r.mask, r.B_Q, r.B_KV, r.N, r.d, Qb, Kb, Vb, sel, row_step=4)
    for n, (h, b) in enumerate(sel):
        rows = np.arange(0, r.B_Q, 4)
        assert np.array_equal(Os[n, rows], O[h, b * r.B_Q + rows])
        assert np.array_equal(Ls[n, rows], LSE[h, b * r.B_Q + rows])
        assert np.isnan(Os[n, 1]).all()
