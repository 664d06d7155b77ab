"""Offline plan-table compilation (paper Section 5.1, Algorithm 1) for the B200 catalog.

For every profiling case (a seeded synthetic mask with its request parameters) and every
eligible catalog plan: run the plan, validate its output (Algorithm 1, lines 4-6), and record
the median forward latency.  Validation has two parts.  (1) A masked-attention reference:
``validator(req, plan_id, O, LSE) -> bool``, applied to every plan including the key's base
plan.  The default, ``sampled_reference_validator``, recomputes seeded query blocks of every
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
            for cid in cids:
                have = {p for (c, p) in latencies if c == cid}
                candidates = have if candidates is None else candidates & have
            if not candidates:
                continue
            gm = {p: math.exp(sum(math.log(latencies[(c, p)]) for c in cids) / len(cids)) for p in candidates}
            ranked = sorted(candidates, key=lambda p: (gm[p], p))
            table[(key, b)] = ranked + [base_plan[key]]
    return table


def write_table(path: str, table: Dict, catalog_hash: int, gpu_name: str, notes: Iterable[str] = ()):
    """Regime line: ``regime B_Q B_KV d nb hb db sb rb : ranked plan ids``."""
    with open(path, "w") as f:
        f.write("BSA_LUT 1\n")
        f.write(f"catalog {catalog_hash:x}\n")
        f.write(f"gpu {gpu_name}\n")
        for n in notes:
            f.write(f"# {n}\n")
        for (key, bucket), ranked in sorted(table.items()):
            f.write("regime " + " ".join(str(x) for x in tuple(key) + tuple(bucket)) + " : " +
                    " ".join(str(p) for p in ranked) + "\n")


# --------------------------------------------------------------------------------------------
# profiling corpus
# --------------------------------------------------------------------------------------------
def corpus(scale: str = "full"):
    """Seeded requests shaped like the five evaluation configurations (seeds >= 1000)."""
    from . import inputs as I
    reqs = []
    nseed = 1 if scale == "quick" else 2
    for s in range(nseed):
        reqs.append(I.config_tiny(seed=1000 + s))
        reqs.append(I.config_mid(seed=1010 + s))
        reqs.append(I.config_stress_b(seed=1030 + s))
        r = I.config_stress_a(seed=1040 + s)
        reqs.append(r)
    reqs.append(I.config_hunyuan(seed=1020))
    if scale != "quick":
        # the same shapes with few heads (head bucket <= 4): what a head-sharded or head-pipelined request looks like
        for n, h in enumerate((1, 2, 3, 4)):
            reqs.append(I.config_mid(seed=1050 + n, H=h))
        reqs.append(I.config_hunyuan(seed=1060, H=3))
        k = 0
        for B in I.SWEEP_GEOMETRIES:
            for rho in I.SWEEP_DENSITIES:
                reqs.append(I.config_sweep(1000 + k, B=B, rho=rho))
                k += 1
    for n, r in enumerate(reqs):
        r.name = f"{r.name}#{n}"
        r.qkv_seed = 5000 + n
    return reqs


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

    def validate(req, plan_id, O, LSE, qkv=None):
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

    validate.wants_qkv = True
    return validate


def profile(reqs, plans=None, reps: int = 5, warmup: int = 3, log=print, validator=None):
    """Algorithm 1, "Profiling": returns (cases, latencies, buckets, base plans).

    ``validator(req, plan_id, O, LSE) -> bool`` is the masked-attention reference of lines 4-6 (default:
    ``sampled_reference_validator()``); a plan it rejects gets no latency.  If it rejects the key's base plan, the
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
        if getattr(validator, "wants_qkv", False):
            return bool(validator(req, pid, O, L, qkv=qkv))
        return bool(validator(req, pid, O, L))

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


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--out", default=DEFAULT_OUT)
    ap.add_argument("--scale", default="full", choices=["full", "quick"])
    args = ap.parse_args(argv)
    import torch
    from . import bsa
    bsa.lut_clear()
    t0 = time.time()
    reqs = corpus(args.scale)
    print(f"corpus: {len(reqs)} cases ({time.time() - t0:.0f} s to generate)")
    cases, lat, bucket, base = profile(reqs)
    table = compile_table(cases, lat, base, lambda cid: bucket[cid])
    write_table(args.out, table, int(bsa.lib().bsa_catalog_hash()), torch.cuda.get_device_name(0),
                notes=[f"{len(cases)} profiling cases, seeds >= 1000, median of 5 forwards after 3 warm-ups, L2 flushed",
                       "regime B_Q B_KV d floor(log2 N) head-bucket density-bucket skew-bucket runcov-bucket : ranked plans, base last"])
    bsa.lut_load(args.out)
    print(f"wrote {args.out}: {len(table)} regimes in {time.time() - t0:.0f} s")
    return 0


if __name__ == "__main__":
    sys.exit(main())
