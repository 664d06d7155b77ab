"""Offline plan-table compilation (paper Section 5.1, Algorithm 1) for the B200 catalog.

For every profiling case (a seeded synthetic mask with its request parameters) and every
eligible catalog plan: run the plan, validate its output (Algorithm 1, lines 4-6), and record
the median forward latency.  Validation has two parts.  (1) A masked-attention reference:
``validator(req, plan_id, O, LSE, qkv) -> bool`` (``qkv``: the CUDA tensors the plan ran on),
applied to every plan including the key's base plan.  The default, ``sampled_reference_validator``, recomputes seeded query blocks of every
head with plain fp32 torch operations on the expanded token-pair mask (dense scores, softmax,
product with V) and compares O and LSE at the contract tolerances; a caller may pass its own
(the tests pass one built on the CPU oracle).  (2) Agreement with the validated base plan's
output on ALL rows, which extends the sampled check to the rows the reference did not visit.
Cases are grouped by request key (B_Q, B_KV, d), partitioned with the runtime's own feature
schema (``bsa_lut_buckets``), and each bucket gets the plans that are valid on all of its cases,
ranked by geometric-mean latency, ties by plan id, followed by the key's base plan.  The result
is the text file ``bsa_lut_load`` reads.

The profiling corpus uses seeds >= 1000, disjoint from every evaluation seed.

    python -m paper_2609_25869_b200.lut_build --out paper_2609_25869_b200/plan_table_b200.lut
"""
from __future__ import annotations

import argparse
import math
import os
import statistics
import sys
import time
from typing import Callable, Dict, Hashable, Iterable, List, Sequence, Tuple

HERE = os.path.dirname(os.path.abspath(__file__))
DEFAULT_OUT = os.path.join(HERE, "plan_table_b200.lut")

O_TOL, O_MEAN_TOL, LSE_TOL = 2e-2, 2e-3, 1e-3  # validation gate (the contract tolerances)


# --------------------------------------------------------------------------------------------
# Algorithm 1, "Regimes and rankings" (pure host logic; unit-tested on the CPU)
# --------------------------------------------------------------------------------------------
_INDEX: Dict[int, Tuple[int, Dict]] = {}


def _by_case(lat: Dict[Tuple[Hashable, int], float]) -> Dict[Hashable, Dict[int, float]]:
    """``lat`` regrouped as {case id: {plan id: latency}}; built once per dictionary (and again if it has grown)."""
    hit = _INDEX.get(id(lat))
    if hit is None or hit[0] != len(lat):
        idx: Dict[Hashable, Dict[int, float]] = {}
        for (c, p), t in lat.items():
            idx.setdefault(c, {})[p] = t
        _INDEX.clear()  # one table is compiled at a time
        _INDEX[id(lat)] = hit = (len(lat), idx)
    return hit[1]


def compile_table(cases: Sequence[Tuple[Hashable, Hashable]], latencies: Dict[Tuple[Hashable, int], float],
                  base_plan: Dict[Hashable, int], bucket_of: Callable[[Hashable], Hashable]) -> Dict:
    """``cases``: (case id, request key); ``latencies[(case id, plan id)]``: validated median latency
    (missing = failed validation or not eligible).  Returns {(key, bucket): [ranked ids..., base]}."""
    table: Dict = {}
    by_key: Dict[Hashable, List[Hashable]] = {}
    for cid, key in cases:
        by_key.setdefault(key, []).append(cid)
    for key, members in by_key.items():
        buckets: Dict[Hashable, List[Hashable]] = {}
        for cid in members:
            buckets.setdefault(bucket_of(cid), []).append(cid)
        for b, cids in buckets.items():
            candidates = None
            per_case = _by_case(latencies)
            for cid in cids:
                have = set(per_case.get(cid, ()))
                candidates = have if candidates is None else candidates & have
            if not candidates:
                continue
            gm = {p: math.exp(sum(math.log(latencies[(c, p)]) for c in cids) / len(cids)) for p in candidates}
            ranked = sorted(candidates, key=lambda p: (gm[p], p))
            table[(key, b)] = ranked + [base_plan[key]]
    return table


# --------------------------------------------------------------------------------------------
# Second stage with learned thresholds (Section 5.1): a decision tree per request key over the
# continuous request features; its leaves are the regimes.  Pure host logic (unit-tested on the CPU).
# --------------------------------------------------------------------------------------------
TREE_FEATURES = ("log2_N", "heads", "density", "skew", "run_coverage")  # indices as the runtime reads them


def case_features(N: int, heads: int, density: float, skew: float, run_coverage: float) -> Tuple[float, ...]:
    return (math.log2(max(1, N)), float(heads), float(density), float(skew), float(run_coverage))


def _case_best(cid, lat) -> float:
    ts = _by_case(lat).get(cid)
    return min(ts.values()) if ts else float("nan")


def _ranking_and_loss(cids, lat, base: int):
    """Ranking of a leaf as in Algorithm 1, lines 15-19 (plans valid on every case of the leaf by geometric-mean
    latency, ties by id, base plan last) and the leaf's loss: the summed log-regret of its cases under the ranking's
    head (a case the head has no latency for falls through the ranking like the runtime's ranked fallback; one that no
    ranked plan serves is charged its slowest measured plan)."""
    cand = None
    per_case = _by_case(lat)
    for c in cids:
        have = set(per_case.get(c, ()))
        cand = have if cand is None else cand & have
    cand = cand or set()
    gm = {p: math.exp(sum(math.log(lat[(c, p)]) for c in cids) / len(cids)) for p in cand}
    ranked = sorted(cand, key=lambda p: (gm[p], p)) + [base]
    return ranked, sum(case_log_regret(c, ranked, lat) for c in cids)


def case_log_regret(cid, ranked, lat) -> float:
    best = _case_best(cid, lat)
    if not best == best:   # no measurement at all for this case
        return 0.0
    for p in ranked:
        if (cid, p) in lat:
            return math.log(lat[(cid, p)] / best)
    return math.log(max(_by_case(lat)[cid].values()) / best)


def learn_tree(cids, feats, lat, base: int, min_leaf: int = 8, max_depth: int = 3):
    """Greedy binary tree: at every node the (feature, threshold) whose two children have the smallest summed loss,
    thresholds taken half-way between neighbouring distinct feature values, both children at least ``min_leaf`` cases;
    a node stays a leaf when no split lowers its loss.  Returns nodes in pre-order (children after their parent):
    ``{"feature": f, "threshold": t, "left": i, "right": j}`` or ``{"ranked": [...], "cases": n}``."""
    nodes: List[dict] = []

    def build(members, depth):
        idx = len(nodes)
        nodes.append({})
        ranked, loss = _ranking_and_loss(members, lat, base)
        best = None
        if depth < max_depth and len(members) >= 2 * min_leaf:
            for f in range(len(TREE_FEATURES)):
                order = sorted(members, key=lambda c: (feats[c][f], str(c)))
                vals = [feats[c][f] for c in order]
                for k in range(min_leaf, len(order) - min_leaf + 1):
                    if vals[k] == vals[k - 1]:
                        continue
                    thr = 0.5 * (vals[k] + vals[k - 1])
                    lo, hi = order[:k], order[k:]
                    total = _ranking_and_loss(lo, lat, base)[1] + _ranking_and_loss(hi, lat, base)[1]
                    if best is None or total < best[0] - 1e-12:
                        best = (total, f, thr, lo, hi)
        if best is not None and best[0] < loss - 1e-9:
            _, f, thr, lo, hi = best
            nodes[idx] = {"feature": f, "threshold": thr}
            nodes[idx]["left"] = build(lo, depth + 1)
            nodes[idx]["right"] = build(hi, depth + 1)
        else:
            nodes[idx] = {"ranked": ranked, "cases": len(members)}
        return idx

    build(list(cids), 0)
    return nodes


def tree_leaf(nodes, feat) -> dict:
    n = nodes[0]
    while "ranked" not in n:
        n = nodes[n["left"] if feat[n["feature"]] < n["threshold"] else n["right"]]
    return n


def choose_depth(cids, feats, groups, lat, base: int, min_leaf: int = 8, depths=(0, 1, 2, 3, 4), folds: int = 4):
    """Tree depth by grouped cross-validation (Section 5.1: masks from the same source stay in one fold): the depth
    with the smallest mean held-out log-regret, the smaller depth on ties.  Returns (depth, {depth: mean log-regret})."""
    names = sorted({groups[c] for c in cids}, key=str)
    fold_of = {g: i % folds for i, g in enumerate(names)}
    score = {}
    for D in depths:
        tot, n = 0.0, 0
        for f in range(min(folds, len(names))):
            train = [c for c in cids if fold_of[groups[c]] != f]
            held = [c for c in cids if fold_of[groups[c]] == f]
            if not train or not held:
                continue
            tree = learn_tree(train, feats, lat, base, min_leaf, D)
            for c in held:
                tot += case_log_regret(c, tree_leaf(tree, feats[c])["ranked"], lat)
                n += 1
        score[D] = tot / max(1, n)
    best = min(score, key=lambda D: (round(score[D], 9), D))
    return best, score


def compile_trees(cases, feats, groups, lat, base_plan, min_leaf: int = 8, max_depth: int = 4, folds: int = 4, log=None):
    """One tree per request key that has at least ``min_leaf`` cases (a single leaf, i.e. one ranking for the key, unless
    it has the ``2 * min_leaf`` a split needs); the other keys keep the fixed-edge regimes alone."""
    by_key: Dict[Hashable, List[Hashable]] = {}
    for cid, key in cases:
        by_key.setdefault(key, []).append(cid)
    trees = {}
    for key, members in sorted(by_key.items()):
        if len(members) < min_leaf:
            continue
        depth, score = choose_depth(members, feats, groups, lat, base_plan[key], min_leaf, tuple(range(max_depth + 1)), folds)
        trees[key] = learn_tree(members, feats, lat, base_plan[key], min_leaf, depth)
        if log:
            log(f"tree {key}: {len(members)} cases, depth {depth} chosen from held-out regret "
                + ", ".join(f"{D}: {math.exp(v):.4f}" for D, v in sorted(score.items()))
                + f"; {sum(1 for n in trees[key] if 'ranked' in n)} leaves")
    return trees


def write_table(path: str, table: Dict, catalog_hash: int, gpu_name: str, notes: Iterable[str] = (), trees: Dict = None):
    """Regime line: ``regime B_Q B_KV d nb hb db sb rb : ranked plan ids``; with ``trees`` the file is version 2 and
    carries, per request key, ``tree B_Q B_KV d n`` followed by its ``node`` lines (pre-order, node 0 the root)."""
    with open(path, "w") as f:
        f.write(f"BSA_LUT {2 if trees else 1}\n")
        f.write(f"catalog {catalog_hash:x}\n")
        f.write(f"gpu {gpu_name}\n")
        for n in notes:
            f.write(f"# {n}\n")
        for (key, bucket), ranked in sorted(table.items()):
            f.write("regime " + " ".join(str(x) for x in tuple(key) + tuple(bucket)) + " : " +
                    " ".join(str(p) for p in ranked) + "\n")
        for key, nodes in sorted((trees or {}).items()):
            f.write("tree " + " ".join(str(x) for x in key) + f" {len(nodes)}\n")
            for i, n in enumerate(nodes):
                if "ranked" in n:
                    f.write(f"node {i} leaf : " + " ".join(str(p) for p in n["ranked"]) + "\n")
                else:
                    f.write(f"node {i} split {n['feature']} {n['threshold']!r} {n['left']} {n['right']}\n")


# --------------------------------------------------------------------------------------------
# profiling corpus
# --------------------------------------------------------------------------------------------
def corpus_specs(scale: str = "full"):
    """The profiling corpus as (generator name, keyword arguments, source group) triples: the five evaluation
    generators with seeds >= 1000 and with head counts, token counts and densities spread over and BETWEEN the values
    the evaluation configurations use, several cases per request key and regime.  ``source group`` names the mask
    source for grouped cross-validation (cases that differ only in head count or seed offset share a source)."""
    specs = []

    def add(gen, group, **kw):
        specs.append((gen, kw, group))

    if scale == "quick":
        for s in range(2):
            add("tiny", f"tiny{s}", seed=1000 + s)
        add("mid", "mid0", seed=1010)
        add("stress_b", "sb0", seed=1030, H=4, N=8192)
        return specs
    # Every request key gets at least 64 cases, so that a tree with the paper's 32 cases per leaf can split it.
    # (64,64) d=64: Tiny's key
    n = 0
    for N in (1024, 2048, 4096, 8192):
        for H, p in ((2, 0.25), (4, 0.1), (8, 0.4), (16, 0.05)):
            for rep in range(4):
                add("tiny", f"tiny{n // 2}", seed=1000 + n, H=H, N=N, p=p * (1.0 + 0.15 * rep))
                n += 1
    # (128,128) d=128: Mid and Hunyuan shapes, and the sweep's (128,128) requests
    n = 0
    for H in (1, 2, 4, 8, 16, 24):
        for extra, win in ((0.02, (1, 1, 1)), (0.0, (1, 1, 1)), (0.1, (1, 1, 1)), (0.02, (2, 1, 1)), (0.3, (0, 0, 0)),
                           (0.05, (1, 1, 1)), (0.01, (1, 2, 2)), (0.2, (1, 0, 0)), (0.5, (0, 0, 0)), (0.0, (2, 2, 2))):
            add("mid", f"mid{n // 2}", seed=1100 + n, H=H, extra=extra, win=win)
            n += 1
    n = 0
    for H in (3, 6, 12, 24):
        for extra, win in ((0.03, (1, 1, 2)), (0.0, (1, 1, 2)), (0.08, (1, 1, 1)), (0.01, (2, 2, 2))):
            add("hunyuan", f"hy{n // 2}", seed=1200 + n, H=H, extra=extra, win=win)
            n += 1
    # (16,64) and (256,256) d=64: the two stress keys
    n = 0
    for N, H in ((8192, 16), (16384, 8), (32768, 16), (32768, 4)):
        for dens in (0.03, 0.05, 0.07, 0.1, 0.15, 0.2, 0.3, 0.4):
            for rep in range(2):
                add("stress_a", f"sa{n // 2}", seed=1300 + n, H=H, N=N, density=dens)
                add("stress_b", f"sb{n // 2}", seed=1400 + n, H=H, N=N, p=min(0.6, dens * 1.4))
                n += 1
    # the sweep's five geometries (d=128, N=75600), densities on and between the sweep's targets
    n = 0
    for H in (3, 6, 12, 24):  # head count outermost: the cases of one shape follow each other and share their tensors
        for B in ((32, 32), (64, 128), (128, 64), (128, 128), (256, 256)):
            for rho in (0.03, 0.05, 0.08, 0.1, 0.17, 0.3, 0.45, 0.6):
                for rep in range(2):
                    add("sweep", f"sw{B[0]}x{B[1]}@{rho}#{rep}", r=1000 + n, H=H, B=B, rho=rho)
                    n += 1
    return specs


def make_case(spec):
    """One corpus case from its spec (host only; runs in the generation pool)."""
    from . import inputs as I
    gen, kw, group = spec
    fn = I.config_sweep if gen == "sweep" else I.CONFIGS[gen]
    req = fn(**kw)
    return req, group


def corpus(scale: str = "full"):
    """The corpus as requests (generated in this process): ``(requests, {case name: source group})``."""
    reqs, groups = [], {}
    for n, spec in enumerate(corpus_specs(scale)):
        r, g = make_case(spec)
        r.name = f"{r.name}#{n}"
        r.qkv_seed = 5000 + n
        reqs.append(r)
        groups[r.name] = g
    return reqs, groups


def head_bucket(heads: int) -> int:
    return 0 if heads <= 4 else (1 if heads <= 16 else 2)


def sampled_reference_validator(blocks_per_head: int = 2, seed: int = 4242):
    """The default masked-attention reference of the validation gate: for ``blocks_per_head`` seeded query blocks of
    every head, dense fp32 scores against all keys, the logical mask expanded to token pairs, softmax, product with V
    (plain torch operations on the GPU, no kernel of this library), compared with the plan's O and LSE."""
    import torch
    from . import inputs as I
    cache = {}

    def reference(req, q, k, v):
        key = (req.name, req.qkv_seed)
        if key in cache:
            return cache[key]
        cache.clear()
        n_kv = req.n_kv
        smp = I.sample_query_blocks(seed, req.H, req.nQb, min(blocks_per_head, req.nQb))
        mask = torch.from_numpy(req.mask).cuda()
        out = []
        was = torch.backends.cuda.matmul.allow_tf32
        torch.backends.cuda.matmul.allow_tf32 = False
        try:
            for h in range(req.H):
                kf, vf = k[h].float(), v[h].float()
                for b in smp[h]:
                    b = int(b)
                    r0, r1 = b * req.B_Q, min(req.N, (b + 1) * req.B_Q)
                    s = (q[h, r0:r1].float() @ kf.T) * (1.0 / req.d ** 0.5)
                    reach = (mask[h, b] != 0).repeat_interleave(req.B_KV)[:n_kv]
                    s = s.masked_fill(~reach[None, :], float("-inf"))
                    lse = torch.logsumexp(s, dim=1)
                    p = torch.exp(s - torch.where(torch.isfinite(lse), lse, torch.zeros_like(lse))[:, None])
                    out.append((h, r0, r1, p @ vf, lse))
        finally:
            torch.backends.cuda.matmul.allow_tf32 = was
        cache[key] = out
        return out

    def validate(req, plan_id, O, LSE, qkv):
        q, k, v = qkv
        err_o, n_o, max_o, max_l = 0.0, 0, 0.0, 0.0
        for h, r0, r1, refO, refL in reference(req, q, k, v):
            fin = torch.isfinite(refL)
            if not torch.equal(torch.isfinite(LSE[h, r0:r1]), fin) or torch.isnan(LSE[h, r0:r1]).any():
                return False
            dO = (O[h, r0:r1].float() - refO).abs()
            if torch.isnan(dO).any():
                return False
            err_o += float(dO.sum())
            n_o += dO.numel()
            max_o = max(max_o, float(dO.max()))
            if fin.any():
                max_l = max(max_l, float((LSE[h, r0:r1][fin] - refL[fin]).abs().max()))
        return max_o <= O_TOL and err_o / max(1, n_o) <= O_MEAN_TOL and max_l <= LSE_TOL

    return validate


def profile(reqs, plans=None, reps: int = 5, warmup: int = 3, log=print, validator=None, features_out=None):
    """Algorithm 1, "Profiling": returns (cases, latencies, buckets, base plans).

    ``validator(req, plan_id, O, LSE, qkv) -> bool`` is the masked-attention reference of lines 4-6 (default:
    ``sampled_reference_validator()``); ``qkv`` are the CUDA tensors the plan ran on (cases of one shape share
    them).  A plan it rejects gets no latency.  ``features_out`` (a dict) receives the continuous request features of
    every case (``case_features``), which the tree compiler partitions on.  ``reqs`` may be any iterable (a generator
    that produces the cases while earlier ones are profiled).  If it rejects the key's base plan, the
    case has no trusted full-size output to compare the other plans with and every plan is judged by it alone."""
    import torch
    from . import bsa
    if validator is None:
        validator = sampled_reference_validator()
    cat = bsa.catalog()
    plan_ids = [c["plan_id"] for c in cat] if plans is None else list(plans)
    cases, lat, bucket, base = [], {}, {}, {}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    qkv_cache = {}

    def passes(req, pid, O, L, qkv):
        return bool(validator(req, pid, O, L, qkv))

    for req in reqs:
        key = (req.B_Q, req.B_KV, req.d)
        shape = (req.H, req.N, req.d)  # tensors are shared by the cases of one shape; the masks differ
        if shape not in qkv_cache:
            qkv_cache.clear()
            qkv_cache[shape] = tuple(t.cuda() for t in req.qkv())
        q, k, v = qkv_cache[shape]
        mask = torch.from_numpy(req.mask).cuda()
        bp = bsa.lib().bsa_base_plan(req.B_Q, req.B_KV, req.d)
        base[key] = bp
        with bsa.plan_create(mask, req.B_Q, req.B_KV, req.N, req.H, req.d, plan_id=bp) as plan:
            refO, refL = plan.forward(q, k, v)
            torch.cuda.synchronize()
            inf = plan.info()
        base_ok = inf["device_status"] == 0 and passes(req, bp, refO, refL, (q, k, v))
        if not base_ok:
            log(f"  base plan {bp} failed validation on {req.name}")
        bk = tuple(inf["regime_bucket"])
        bucket[req.name] = (bk[0], head_bucket(req.H), bk[1], bk[2], bk[3])
        if features_out is not None:
            features_out[req.name] = case_features(req.N, req.H, inf["density"], inf["skew"], inf["run_coverage"])
        cases.append((req.name, key))
        fin = torch.isfinite(refL)
        row = []
        for pid in plan_ids:
            if not bsa.plan_eligible(pid, req.B_Q, req.B_KV, req.N, req.H, req.d):
                continue
            with bsa.plan_create(mask, req.B_Q, req.B_KV, req.N, req.H, req.d, plan_id=pid) as plan:
                O, L = plan.forward(q, k, v)
                torch.cuda.synchronize()
                ok = plan.info()["device_status"] == 0
                ok = ok and (base_ok if pid == bp else passes(req, pid, O, L, (q, k, v)))
                if ok and base_ok and pid != bp:  # all rows against the validated base plan's output
                    ok = bool(torch.equal(torch.isfinite(L), fin))
                    ok = ok and float((O.float() - refO.float()).abs().max()) <= O_TOL
                    ok = ok and (not fin.any() or float((L[fin] - refL[fin]).abs().max()) <= LSE_TOL)
                if not ok:
                    log(f"  plan {pid} failed validation on {req.name}")
                    continue
                for _ in range(warmup):
                    plan.forward(q, k, v, O, L)
                ts = []
                for i in range(reps):
                    flush.fill_(i)
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record()
                    plan.forward(q, k, v, O, L)
                    b.record()
                    b.synchronize()
                    ts.append(a.elapsed_time(b))
                lat[(req.name, pid)] = statistics.median(ts)
                row.append((lat[(req.name, pid)], pid))
        row.sort()
        log(f"{req.name:14s} key={key} bucket={bucket[req.name]} density={inf['density']:.3f} skew={inf['skew']:.2f} "
            f"best: " + ", ".join(f"{cat[p]['name']}={t * 1e3:.0f}us" for t, p in row[:3]))
    return cases, lat, bucket, base


def leave_source_out(path: str, min_leaf: int = 32, max_depth: int = 4, log=print) -> Dict[str, dict]:
    """Offline check of how the table generalises, from a latencies file written by ``--latencies``: every mask source
    in turn is left out of the corpus, regimes and trees are compiled from the rest, and each left-out case is looked
    up in them in three ways (regimes then trees then base plan, as the runtime does; trees alone; regimes alone).
    Returns per way the geometric-mean regret, the share within 3 % and the share of cases that found a regime or leaf.
    Needs the library only for the fixed-edge bucket function and the base plans (no GPU)."""
    import ctypes
    import json
    from . import bsa
    with open(path) as f:
        d = json.load(f)
    cases = [(c, tuple(k)) for c, k in d["cases"]]
    lat = {(c, int(pid)): t for c, pid, t in d["lat"]}
    feats = {c: tuple(v) for c, v in d["features"].items()}
    groups = d["groups"]
    lib = bsa.lib()
    lib.bsa_lut_buckets.argtypes = [ctypes.c_int64, ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                    ctypes.POINTER(ctypes.c_int32)]
    lib.bsa_lut_buckets.restype = None
    bucket, base = {}, {}
    for c, key in cases:
        lg, heads, dens, skew, rc = feats[c]
        out = (ctypes.c_int32 * 4)()
        lib.bsa_lut_buckets(int(round(2.0 ** lg)), dens, skew, rc, out)
        bucket[c] = (out[0], head_bucket(int(heads)), out[1], out[2], out[3])
        base[key] = int(lib.bsa_base_plan(key[0], key[1], key[2]))
    sources = sorted(set(groups.values()))
    acc = {w: {"log": 0.0, "n": 0, "within": 0, "found": 0} for w in ("regime_tree_base", "tree_base", "regime_base")}
    for src in sources:
        held = [(c, k) for c, k in cases if groups[c] == src]
        keys = {k for _, k in held}  # only the tables of the left-out cases' own request keys matter
        train = [(c, k) for c, k in cases if groups[c] != src and k in keys]
        table = compile_table(train, lat, base, lambda cid: bucket[cid])
        trees = compile_trees(train, feats, groups, lat, base, min_leaf=min_leaf, max_depth=max_depth)
        for c, key in held:
            reg = table.get((key, bucket[c]))
            leaf = tree_leaf(trees[key], feats[c])["ranked"] if key in trees else None
            for way, ranked in (("regime_tree_base", reg or leaf), ("tree_base", leaf), ("regime_base", reg)):
                a = acc[way]
                lr = case_log_regret(c, ranked if ranked else [base[key]], lat)
                a["log"] += lr
                a["n"] += 1
                a["within"] += 1 if lr <= math.log(1.03) else 0
                a["found"] += 1 if ranked else 0
    res = {}
    for way, a in acc.items():
        res[way] = {"cases": a["n"], "regret_gm": math.exp(a["log"] / max(a["n"], 1)),
                    "within_3pct": a["within"] / max(a["n"], 1), "found": a["found"] / max(a["n"], 1)}
        if log:
            log(f"{way}: {res[way]}")
    return res


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--leave-source-out", default="", metavar="LATENCIES.json",
                    help="no profiling: leave every mask source out of the recorded corpus in turn and report the regret "
                    "of the left-out cases (host only)")
    ap.add_argument("--out", default=DEFAULT_OUT)
    ap.add_argument("--scale", default="full", choices=["full", "quick"])
    ap.add_argument("--min-leaf", type=int, default=32, help="fewest cases a tree leaf may hold (Section 5.1: 32)")
    ap.add_argument("--max-depth", type=int, default=4)
    ap.add_argument("--no-trees", action="store_true", help="fixed-edge regimes only")
    ap.add_argument("--latencies", default="", help="also write the measured latencies as JSON (for the regret report)")
    args = ap.parse_args(argv)
    if args.leave_source_out:
        leave_source_out(args.leave_source_out, args.min_leaf, args.max_depth)
        return 0
    specs = corpus_specs(args.scale)
    # masks are generated by worker processes (forked before CUDA is touched) while earlier cases are profiled
    import multiprocessing as mp
    pool = mp.get_context("fork").Pool(max(1, min(12, (os.cpu_count() or 2) - 2)))
    stream = pool.imap(make_case, specs)
    import torch
    from . import bsa
    bsa.lut_clear()
    t0 = time.time()
    groups = {}

    def cases_in_order():
        for n, (req, group) in enumerate(stream):
            req.name = f"{req.name}#{n}"
            req.qkv_seed = 5000 + n
            groups[req.name] = group
            yield req

    print(f"corpus: {len(specs)} cases")
    feats = {}
    cases, lat, bucket, base = profile(cases_in_order(), features_out=feats)
    pool.terminate()
    table = compile_table(cases, lat, base, lambda cid: bucket[cid])
    trees = {} if args.no_trees else compile_trees(cases, feats, groups, lat, base, min_leaf=args.min_leaf,
                                                   max_depth=args.max_depth, log=print)
    write_table(args.out, table, int(bsa.lib().bsa_catalog_hash()), torch.cuda.get_device_name(0),
                notes=[f"{len(cases)} profiling cases, seeds >= 1000, median of 5 forwards after 3 warm-ups, L2 flushed",
                       "regime B_Q B_KV d floor(log2 N) head-bucket density-bucket skew-bucket runcov-bucket : ranked plans, base last",
                       f"tree features: {' '.join(TREE_FEATURES)}; a key with a tree is looked up there, the others in the regimes"],
                trees=trees)
    if args.latencies:
        import json
        with open(args.latencies, "w") as f:
            json.dump({"cases": [[c, list(k)] for c, k in cases], "lat": [[c, p, t] for (c, p), t in lat.items()],
                       "features": feats, "groups": groups}, f)
    bsa.lut_load(args.out)
    print(f"wrote {args.out}: {len(table)} regimes, {len(trees)} trees in {time.time() - t0:.0f} s")
    return 0


if __name__ == "__main__":
    sys.exit(main())
