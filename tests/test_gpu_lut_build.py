"""Offline plan-table compilation (Algorithm 1) on the GPU: profiling with a validation gate built on the CPU oracle,
ranking, the written file, and the online lookup (Algorithm 2) that reads it back."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_25869_b200 import bsa, lut_build
from paper_2609_25869_b200 import inputs as I
from tests import helpers as Hh

pytestmark = pytest.mark.gpu


def _oracle_validator(corrupt=None):
    """validator(req, plan_id, O, LSE, qkv): 8 seeded query blocks per head against the fp64 oracle (on the tensors the
    plan ran on) at the contract tolerances.  `corrupt` = (case name, plan id): that plan's output is damaged before
    it is validated."""
    cache = {}

    def validate(req, plan_id, O, LSE, qkv):
        if req.name not in cache:
            Qb, Kb, Vb = (I.bf16_bits(t.cpu()) for t in qkv)
            smp = I.sample_query_blocks(5, req.H, req.nQb, min(8, req.nQb))
            sel = [(h, int(b)) for h in range(req.H) for b in smp[h]]
            cache[req.name] = (sel,) + tuple(oracle.attention_blocks(req.mask, req.B_Q, req.B_KV, req.N, req.d, Qb, Kb, Vb, sel)[:2])
        sel, refO, refL = cache[req.name]
        O = O.float().cpu().numpy().copy()
        LSE = LSE.cpu().numpy()
        if corrupt == (req.name, plan_id):
            h, b = sel[0]
            O[h, b * req.B_Q] += 0.25           # one row of one sampled block
        dO, dL = [], []
        for n, (h, b) in enumerate(sel):
            r0 = b * req.B_Q
            rows = min(req.B_Q, req.N - r0)
            fin = np.isfinite(refL[n, :rows])
            if not np.array_equal(np.isfinite(LSE[h, r0:r0 + rows]), fin):
                return False
            dO.append(np.abs(O[h, r0:r0 + rows] - refO[n, :rows]).ravel())
            dL.append(np.abs(LSE[h, r0:r0 + rows][fin] - refL[n, :rows][fin]))
        dO, dL = np.concatenate(dO), np.concatenate(dL)
        return bool(dO.max() <= Hh.O_MAX_ABS and dO.mean() <= Hh.O_MEAN_ABS and (dL.size == 0 or dL.max() <= Hh.LSE_ABS))

    return validate


@pytest.fixture
def _restore_table():
    yield
    bsa.lut_clear()
    bsa.load_default_table()


def _quick_corpus():
    reqs = [I.config_tiny(seed=1000), I.config_tiny(seed=1001), I.config_mid(seed=1010, H=2)]
    for n, r in enumerate(reqs):
        r.name = f"{r.name}#{n}"
        r.qkv_seed = 5000 + n
    return reqs


def test_profile_validates_against_the_oracle_and_the_table_selects_the_fastest_valid_plan(tmp_path, _restore_table):
    bsa.lut_clear()
    reqs = _quick_corpus()
    plans = [0, 22, 23, 25, 27]
    bad = (reqs[0].name, 23)
    log = []
    cases, lat, bucket, base = lut_build.profile(reqs, plans=plans, reps=3, warmup=2, log=log.append,
                                                 validator=_oracle_validator(corrupt=bad))
    # Algorithm 1, lines 4-9: the corrupted candidate has no latency, every other eligible plan has one
    assert bad not in lat and any("plan 23 failed validation" in l for l in log)
    for r in reqs:
        for pid in plans:
            assert ((r.name, pid) in lat) == ((r.name, pid) != bad), (r.name, pid)
    assert all(t > 0 for t in lat.values())
    # lines 10-19: ranking per bucket over the plans valid on all of its cases, base plan appended
    table = lut_build.compile_table(cases, lat, base, lambda cid: bucket[cid])
    tiny_key = (reqs[0].B_Q, reqs[0].B_KV, reqs[0].d)
    b0 = bucket[reqs[0].name]
    assert 23 not in table[(tiny_key, b0)][:-1]
    if bucket[reqs[1].name] != b0:                       # the other Tiny case may or may not share the bucket
        assert 23 in table[(tiny_key, bucket[reqs[1].name])]
    path = str(tmp_path / "quick.lut")
    lut_build.write_table(path, table, int(bsa.lib().bsa_catalog_hash()), "test")
    bsa.lut_load(path)
    assert bsa.lib().bsa_lut_num_regimes() == len(table)
    # Algorithm 2, lines 6-14: a corpus case looked up online gets the head of its regime's ranking, which is the
    # valid plan with the smallest geometric-mean latency over the regime's cases
    for r in reqs:
        key, b = (r.B_Q, r.B_KV, r.d), bucket[r.name]
        members = [c for c, k in cases if k == key and bucket[c] == b]
        valid = [p for p in plans if all((c, p) in lat for c in members)]
        gm = {p: float(np.exp(np.mean([np.log(lat[(c, p)]) for c in members]))) for p in valid}
        want = min(valid, key=lambda p: (gm[p], p))
        assert table[(key, b)][0] == want and table[(key, b)][-1] == base[key]
        with bsa.plan_create(torch.from_numpy(r.mask).cuda(), r.B_Q, r.B_KV, r.N, r.H, r.d) as plan:
            inf = plan.info()
        assert inf["lut_hit"] == 1 and inf["plan"]["plan_id"] == want


def test_default_reference_of_the_validation_gate_accepts_a_plan_and_rejects_damage():
    """The gate's default masked-attention reference (plain torch operations on the expanded mask): it accepts the
    outputs of two kernel families on a ragged request and rejects a shifted output row, a wrong LSE and an LSE
    that is finite on an empty row."""
    M = I.random_mask(7, 2, I.cdiv(1000, 64), I.cdiv(1000, 32), 0.3, diag=True, empty_rows=0.2)
    req = I.Request("gate", 2, 1000, 64, 64, 32, M, qkv_seed=3)
    mask, q, k, v, _ = Hh.to_dev(req)
    val = lut_build.sampled_reference_validator(blocks_per_head=req.nQb)   # every block
    for pid in (22, 1):
        with bsa.plan_create(mask, req.B_Q, req.B_KV, req.N, req.H, req.d, plan_id=pid) as plan:
            O, L = plan.forward(q, k, v)
            torch.cuda.synchronize()
        assert val(req, pid, O, L, (q, k, v))
    row = int(np.flatnonzero(M[0].sum(axis=1) > 0)[0]) * 64
    O2 = O.clone(); O2[0, row] += 0.1
    L2 = L.clone(); L2[0, row] += 0.01
    assert not val(req, 1, O2, L, (q, k, v)) and not val(req, 1, O, L2, (q, k, v))
    empty = np.flatnonzero(M[1].sum(axis=1) == 0)
    assert len(empty)
    L3 = L.clone(); L3[1, int(empty[0]) * 64] = 0.0
    assert not val(req, 1, O, L3, (q, k, v))
