"""CPU-only tests: the C-ABI library loads and exports what include/bsa.h declares, the catalog and
eligibility rules, and the plan-table lookup (Algorithm 2) against the oracle's restatement of it."""
import ctypes
import os
import re
import subprocess

import numpy as np
import pytest

from oracle import oracle
from paper_2609_25869_b200 import bsa
from paper_2609_25869_b200 import build as bsa_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    bsa_build.build()
    bsa.lut_clear()
    yield
    bsa.lut_clear()


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "bsa.h")).read()
    declared = set(re.findall(r"BSA_API\s+[\w\s\*]+?\b(bsa_\w+)\s*\(", hdr))
    assert {"bsa_plan_create", "bsa_forward", "bsa_plan_destroy"} <= declared and len(declared) >= 20
    out = subprocess.check_output(["nm", "-D", "--defined-only", bsa.LIB_PATH], text=True)
    exported = set(l.split()[-1] for l in out.splitlines() if " T " in l)
    assert declared <= exported, declared - exported
    assert all(s.startswith("bsa_") for s in exported), "only the C ABI is exported"
    L = bsa.lib()
    for name in declared:
        assert hasattr(L, name)


def test_catalog_and_eligibility():
    cat = bsa.catalog()
    assert len(cat) >= 6 and [c["plan_id"] for c in cat] == list(range(len(cat)))
    assert len(set(c["name"] for c in cat)) == len(cat)
    assert {c["T_KV"] for c in cat} == {16, 32, 64, 128} and {c["T_Q"] for c in cat} == {16, 128, 256}
    assert {c["kernel"] for c in cat} == {0, 1, 2, 3, 4, 5}
    base = bsa.lib().bsa_base_plan(128, 128, 128)
    # the base plan is eligible for every supported request key
    for B_Q in (16, 32, 64, 128, 256):
        for B_KV in (16, 32, 64, 128, 256):
            for d in (64, 128, 256):
                assert bsa.plan_eligible(bsa.lib().bsa_base_plan(B_Q, B_KV, d), B_Q, B_KV, 75600, 24, d)
    assert not bsa.plan_eligible(base, 8, 64, 1024, 1, 64)       # block size below 16
    assert not bsa.plan_eligible(base, 64, 64, 1024, 1, 96)      # head dim outside the catalog
    assert not bsa.plan_eligible(len(cat), 64, 64, 1024, 1, 64)  # unknown plan
    split = next(c for c in cat if c["split_pmax"] > 1)
    assert bsa.plan_eligible(split["plan_id"], 64, 64, 2048, 2, 64)
    assert not bsa.plan_eligible(split["plan_id"], 64, 64, 2048, 2, 64, max_workspace_bytes=4096)  # workspace
    assert not bsa.plan_eligible(split["plan_id"], 128, 128, 115200, 24, 128)  # default workspace limit
    # the 16-row-tile kernel: logical blocks of up to 64 rows, KV tiles no wider than the block or the staging buffer, bf16
    rb = {c["name"]: c["plan_id"] for c in cat if c["kernel"] == 5}
    assert bsa.plan_eligible(rb["q16k64_rb"], 16, 64, 32768, 16, 64) and bsa.plan_eligible(rb["q16k32_rb"], 32, 32, 75600, 24, 128)
    assert not bsa.plan_eligible(rb["q16k64_rb"], 16, 64, 32768, 16, 128)     # 64 keys x 128 x 2 bytes > 8 KB staging
    assert not bsa.plan_eligible(rb["q16k64_rb"], 16, 32, 32768, 16, 64)      # would need membership masks
    assert not bsa.plan_eligible(rb["q16k32_rb"], 128, 128, 16384, 8, 128)    # nothing to win on 128-row blocks
    # half tensors: every kernel family but the paired (ids 10-13) and the column-split one (14-17)
    assert bsa.plan_eligible(rb["q16k32_rb"], 32, 32, 75600, 24, 128, dtype="fp16")
    assert bsa.plan_eligible(22, 128, 128, 4096, 2, 128, N_kv=999, dtype="fp16") and bsa.plan_eligible(0, 128, 128, 4096, 2, 128, dtype="fp16")
    assert not bsa.plan_eligible(10, 128, 128, 4096, 2, 128, dtype="fp16") and not bsa.plan_eligible(14, 128, 128, 4096, 2, 128, dtype="fp16")
    assert bsa.plan_eligible(19, 128, 128, 4096, 2, 256, dtype="fp16") and not bsa.plan_eligible(22, 128, 128, 4096, 2, 256, dtype="fp16")


def test_feature_schema_buckets():
    assert bsa.lut_buckets(16384, 0.15, 1.5, 0.8) == [14, 4, 1, 1]
    assert bsa.lut_buckets(16383, 0.0199, 1.49, 0.49) == [13, 0, 0, 0]
    assert bsa.lut_buckets(115200, 0.9, 100.0, 1.0) == [16, 6, 3, 1]


def _write_lut(path, regimes, catalog_hash=None, version=1):
    h = bsa.lib().bsa_catalog_hash() if catalog_hash is None else catalog_hash
    with open(path, "w") as f:
        f.write(f"BSA_LUT {version}\ncatalog {h:x}\ngpu test\n")
        for key, ids in regimes.items():
            f.write("regime " + " ".join(str(x) for x in key) + " : " + " ".join(str(i) for i in ids) + "\n")


def test_plan_table_lookup_matches_algorithm_2(tmp_path):
    # regime key: B_Q B_KV d floor(log2 N) head-bucket density-bucket skew-bucket runcov-bucket
    regimes = {
        (64, 64, 64, 11, 0, 5, 1, 0): [3, 1, 0],
        (128, 128, 128, 16, 2, 2, 0, 1): [2, 1, 0],   # plan 2 needs a workspace this request cannot bind
    }
    p = str(tmp_path / "t.lut")
    _write_lut(p, regimes)
    bsa.lut_load(p)
    assert bsa.lib().bsa_lut_num_regimes() == 2
    BASE = bsa.lib().bsa_base_plan(64, 64, 64)
    base = {("k64",): BASE}
    # hit: first eligible plan of the ranking
    pid, hit = bsa.lut_select(64, 64, 2048, 2, 64, 0.27, 0.4, 1.6)
    assert (pid, hit) == (3, True)
    assert pid == oracle.select_plan({(("k64",), "b"): [3, 1, 0]}, base, ("k64",), "b", lambda q: True)
    # ranked fallback: plan 2 is not eligible (workspace over the default limit) -> next in rank order
    pid, hit = bsa.lut_select(128, 128, 115200, 24, 128, 0.066, 0.9, 1.2)
    assert (pid, hit) == (1, True)
    assert pid == oracle.select_plan({(("k",), "b"): [2, 1, 0]}, {("k",): BASE}, ("k",), "b", lambda q: q != 2)
    # miss: the base plan alone
    pid, hit = bsa.lut_select(64, 64, 2048, 2, 64, 0.01, 0.4, 1.6)
    assert (pid, hit) == (BASE, False)
    assert pid == oracle.select_plan({}, base, ("k64",), "other", lambda q: True)
    # nothing eligible -> no-eligible-plan
    pid, hit = bsa.lut_select(64, 64, 2048, 2, 96, 0.27, 0.4, 1.6)
    assert pid == -1
    assert oracle.select_plan({}, base, ("k64",), "other", lambda q: False) is None
    bsa.lut_clear()
    assert bsa.lut_select(64, 64, 2048, 2, 64, 0.27, 0.4, 1.6) == (BASE, False)


def test_plan_table_rejects_foreign_or_malformed_files(tmp_path):
    good = {(64, 64, 64, 11, 0, 5, 1, 0): [1, 0]}
    p = str(tmp_path / "bad.lut")
    _write_lut(p, good, catalog_hash=0x1234)          # built for another catalog
    with pytest.raises(bsa.BsaError) as e:
        bsa.lut_load(p)
    assert e.value.status == 7 and bsa.lib().bsa_lut_num_regimes() == 0
    _write_lut(p, good, version=3)                    # unknown version
    with pytest.raises(bsa.BsaError):
        bsa.lut_load(p)
    _write_lut(p, {(64, 64, 64, 11, 0, 5, 1, 0): [999]})  # unknown plan id
    with pytest.raises(bsa.BsaError):
        bsa.lut_load(p)
    with pytest.raises(bsa.BsaError):
        bsa.lut_load(str(tmp_path / "missing.lut"))
    _write_lut(p, good)
    bsa.lut_load(p)
    assert bsa.lib().bsa_lut_num_regimes() == 1
    bsa.lut_clear()


def test_status_strings_and_version():
    L = bsa.lib()
    assert L.bsa_status_string(0) == b"ok" and L.bsa_status_string(3) == b"no eligible plan"
    assert b"sm_100a" in L.bsa_version()


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(bsa, "_lib", None)
    monkeypatch.setattr(bsa, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        bsa.lib()


def test_offline_table_compilation_matches_algorithm_1(tmp_path):
    """lut_build.compile_table (product) against the oracle's restatement of Algorithm 1, and the
    written file loads back into the runtime with the same rankings."""
    from paper_2609_25869_b200 import lut_build
    import random
    rnd = random.Random(3)
    keys = [(128, 128, 128), (64, 64, 64)]
    cases, lat, bucket = [], {}, {}
    for n in range(24):
        key = keys[n % 2]
        cid = f"case{n}"
        cases.append((cid, key))
        bucket[cid] = (14, 1, n % 3, 0, 1)
        for pid in range(6):
            if rnd.random() < 0.15:
                continue  # failed validation / not eligible on this case
            lat[(cid, pid)] = rnd.choice([1.0, 2.0, 4.0]) * (1 + (pid == 3))
    base = {keys[0]: 0, keys[1]: 1}
    got = lut_build.compile_table(cases, lat, base, bucket.get)
    want = oracle.compile_table(cases, lat, base, bucket.get)
    assert got == want and len(got) >= 4
    for ranked in got.values():
        assert ranked[-1] in (0, 1) and len(set(ranked[:-1])) == len(ranked) - 1
    path = str(tmp_path / "t.lut")
    lut_build.write_table(path, got, int(bsa.lib().bsa_catalog_hash()), "test-gpu")
    bsa.lut_load(path)
    assert bsa.lib().bsa_lut_num_regimes() == len(got)
    bsa.lut_clear()


def test_decision_tree_regimes_hand_built_case(tmp_path):
    """Second stage with learned thresholds (Section 5.1): on a hand-built corpus where plan 1 wins below 20 % density
    and plan 3 above it, whatever the other features, the tree compiler finds one split on density between the two
    clusters, cross-validation (folds by mask source) prefers depth 1 over depth 0, the leaves carry the rankings of
    Algorithm 1 with the base plan last, and the runtime reads the file back and walks the same tree."""
    from paper_2609_25869_b200 import lut_build as LB
    key = (128, 128, 128)
    cases, feats, groups, lat = [], {}, {}, {}
    for n in range(24):
        cid = f"c{n}"
        low = n % 2 == 0
        density = (0.04 + 0.01 * (n % 5)) if low else (0.35 + 0.02 * (n % 7))
        cases.append((cid, key))
        feats[cid] = LB.case_features(16384 if n % 3 else 65536, 8 + (n % 4), density, 1.0 + 0.1 * (n % 6), 0.5)
        groups[cid] = f"source{n // 2}"            # a low and a high case per source
        lat[(cid, 1)] = 1.0 if low else 2.0
        lat[(cid, 3)] = 1.5 if low else 1.0
        lat[(cid, 22)] = 3.0                        # the base plan: valid everywhere, never best
        if n == 5:
            del lat[(cid, 1)]                       # plan 1 failed validation on one high-density case
    base = {key: 22}
    depth, score = LB.choose_depth([c for c, _ in cases], feats, groups, lat, 22, min_leaf=4, depths=(0, 1, 2), folds=4)
    assert depth == 1 and score[1] < score[0] - 0.1 and abs(score[1]) < 1e-12
    trees = LB.compile_trees(cases, feats, groups, lat, base, min_leaf=4, max_depth=2, folds=4)
    t = trees[key]
    assert t[0]["feature"] == 2 and 0.08 < t[0]["threshold"] < 0.35 and len(t) == 3
    lo, hi = t[t[0]["left"]], t[t[0]["right"]]
    assert lo["ranked"] == [1, 3, 22, 22] and lo["cases"] == 12
    assert hi["ranked"] == [3, 22, 22] and hi["cases"] == 12   # plan 1 is not valid on every high-density case
    # with no split allowed the single leaf ranks by geometric mean over everything
    flat = LB.learn_tree([c for c, _ in cases], feats, lat, 22, min_leaf=4, max_depth=0)
    assert len(flat) == 1 and flat[0]["ranked"] == [3, 22, 22]
    # too few cases for two leaves of min_leaf: a single leaf (one ranking for the key); fewer than one leaf's worth: no tree
    single = LB.compile_trees(cases[:6], feats, groups, lat, base, min_leaf=4)
    assert len(single[key]) == 1 and single[key][0]["cases"] == 6 and single[key][0]["ranked"][-1] == 22
    assert LB.compile_trees(cases[:3], feats, groups, lat, base, min_leaf=4) == {}
    path = str(tmp_path / "tree.lut")
    LB.write_table(path, {}, int(bsa.lib().bsa_catalog_hash()), "test", trees=trees)
    bsa.lut_load(path)
    assert bsa.lib().bsa_lut_num_trees() == 1 and bsa.lib().bsa_lut_num_regimes() == 0
    assert bsa.lut_select(128, 128, 16384, 8, 128, 0.05, 0.5, 1.2) == (1, True)
    assert bsa.lut_select(128, 128, 16384, 8, 128, 0.50, 0.5, 1.2) == (3, True)
    assert bsa.lut_select(128, 128, 16384, 8, 128, t[0]["threshold"], 0.5, 1.2) == (3, True)   # feature < threshold goes left
    assert bsa.lut_select(64, 64, 16384, 8, 128, 0.05, 0.5, 1.2) == (bsa.lib().bsa_base_plan(64, 64, 128), False)  # key without a tree
    # a fixed-edge regime of the same key takes precedence where it exists; everywhere else the tree answers
    b = bsa.lut_buckets(16384, 0.05, 1.2, 0.5)
    LB.write_table(path, {(key, (b[0], 1, b[1], b[2], b[3])): [7, 22]}, int(bsa.lib().bsa_catalog_hash()), "test", trees=trees)
    bsa.lut_load(path)
    assert bsa.lut_select(128, 128, 16384, 8, 128, 0.05, 0.5, 1.2) == (7, True)
    assert bsa.lut_select(128, 128, 16384, 8, 128, 0.50, 0.5, 1.2) == (3, True)
    LB.write_table(path, {}, int(bsa.lib().bsa_catalog_hash()), "test", trees=trees)
    # malformed trees are rejected as a whole file
    text = open(path).read()
    for bad in (text.replace("BSA_LUT 2", "BSA_LUT 1"), text.replace("node 2 leaf", "node 1 leaf"),
                text.replace("split 2", "split 9"), text.replace(" 3\nnode 0", " 4\nnode 0")):
        with open(path, "w") as f:
            f.write(bad)
        with pytest.raises(bsa.BsaError):
            bsa.lut_load(path)
        assert bsa.lib().bsa_lut_num_trees() == 0
    bsa.lut_clear()


def test_regret_summary_statistics():
    """Selection-regret summary (host arithmetic only): geometric mean, percentiles, 3 % band for win/tie/loss."""
    from paper_2609_25869_b200.regret import summarise
    rows = [{"t_selected": 1.00, "t_best": 1.00, "t_base": 1.50},   # regret 1.00, speedup 1.50 -> win
            {"t_selected": 2.04, "t_best": 2.00, "t_base": 2.04},   # regret 1.02, speedup 1.00 -> tie
            {"t_selected": 1.10, "t_best": 1.00, "t_base": 1.00},   # regret 1.10, speedup 0.909 -> loss
            {"t_selected": 4.00, "t_best": 4.00, "t_base": 4.10}]   # regret 1.00, speedup 1.025 -> tie
    s = summarise(rows)
    assert s["n"] == 4 and (s["win"], s["tie"], s["loss"]) == (1, 2, 1)
    assert abs(s["regret_gm"] - (1.0 * 1.02 * 1.10 * 1.0) ** 0.25) < 1e-12
    assert s["regret_max"] == 1.10 and s["regret_p95"] == 1.10 and abs(s["within_3pct"] - 0.75) < 1e-12
    assert abs(s["speedup_vs_base_gm"] - (1.5 * 1.0 * (1 / 1.1) * 1.025) ** 0.25) < 1e-12


def test_pack_mask_matches_numpy_packbits():
    """The binding's bit-packing helper: little-endian bits, rows padded to a multiple of 4 bytes."""
    import torch
    rng = np.random.default_rng(3)
    for nk in (1, 7, 8, 31, 32, 33, 100):
        m = (rng.random((2, 5, nk)) < 0.4).astype(np.uint8)
        packed, stride = bsa.pack_mask(torch.from_numpy(m))
        assert stride % 4 == 0 and stride * 8 >= nk and packed.shape == (2, 5, stride)
        ref = np.packbits(m, axis=2, bitorder="little")
        got = packed.numpy()
        assert np.array_equal(got[:, :, : ref.shape[2]], ref) and not got[:, :, ref.shape[2]:].any()


def test_packed_create_rejects_bad_layouts_without_a_gpu():
    h = ctypes.c_void_p()
    L = bsa.lib()
    fake = ctypes.c_void_p(0x1000)  # never dereferenced: the checks come first
    assert L.bsa_plan_create_packed(fake, 6, 128, 128, 1024, 1, 128, None, None, ctypes.byref(h)) == 1   # stride % 4
    assert L.bsa_plan_create_packed(fake, 0, 128, 128, 1024, 1, 128, None, None, ctypes.byref(h)) == 1   # stride <= 0
    assert L.bsa_plan_create_packed(fake, 4, 16, 16, 1024, 1, 128, None, None, ctypes.byref(h)) == 1     # 64 blocks > 32 bits
    assert L.bsa_plan_create_packed(ctypes.c_void_p(0x1002), 8, 16, 16, 1024, 1, 128, None, None, ctypes.byref(h)) == 1
    assert L.bsa_plan_create_packed(None, 8, 16, 16, 1024, 1, 128, None, None, ctypes.byref(h)) == 1


def test_plan_cache_host_calls_without_a_gpu():
    """The cache itself is host state: it is created, read and destroyed without a device, and bad arguments are
    refused before anything touches one."""
    L = bsa.lib()
    c = ctypes.c_void_p()
    assert L.bsa_plan_cache_create(0, ctypes.byref(c)) == 1
    assert L.bsa_plan_cache_create(4, None) == 1
    assert L.bsa_plan_cache_create(4, ctypes.byref(c)) == 0 and c.value
    hits, misses, ev = ctypes.c_int64(-1), ctypes.c_int64(-1), ctypes.c_int64(-1)
    n = ctypes.c_int32(-1)
    assert L.bsa_plan_cache_stats(c, ctypes.byref(hits), ctypes.byref(misses), ctypes.byref(ev), ctypes.byref(n)) == 0
    assert (hits.value, misses.value, ev.value, n.value) == (0, 0, 0, 0)
    h = ctypes.c_void_p()
    fake = ctypes.c_void_p(0x1000)  # never dereferenced: the checks come first
    assert L.bsa_plan_cache_get(None, fake, 0, 128, 128, 1024, 1, 128, None, None, ctypes.byref(h), None) == 1
    assert L.bsa_plan_cache_get(c, fake, -4, 128, 128, 1024, 1, 128, None, None, ctypes.byref(h), None) == 1
    assert L.bsa_plan_cache_get(c, None, 0, 128, 128, 1024, 1, 128, None, None, ctypes.byref(h), None) == 1
    assert L.bsa_plan_cache_get(c, fake, 6, 128, 128, 1024, 1, 128, None, None, ctypes.byref(h), None) == 1   # stride % 4
    assert L.bsa_plan_cache_get(c, fake, 0, 128, 128, 1024, 1, 96, None, None, ctypes.byref(h), None) == 2    # d unsupported
    assert L.bsa_plan_cache_stats(None, None, None, None, None) == 1
    assert L.bsa_plan_cache_destroy(c) == 0
    assert L.bsa_plan_cache_destroy(None) == 1
