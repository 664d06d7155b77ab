"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element, on the
same seeded inputs; the tile plan's coverage against E(M), bit-exact."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_25869_b200 import bsa
from paper_2609_25869_b200 import inputs as I
from tests import helpers as Hh

pytestmark = pytest.mark.gpu


def _sample(req, per_head, seed=77, heads=None):
    smp = I.sample_query_blocks(seed, req.H, req.nQb, per_head)
    hs = range(req.H) if heads is None else heads
    return [(h, int(b)) for h in hs for b in smp[h]]


# ---------------------------------------------------------------- the five configurations
@pytest.mark.parametrize("plan_id", [-1, 0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12, 13, 14, 15, 16, 17, 18, 19, 20, 21, 22, 23, 24, 25, 26, 27, 28, 29, 30, 31, 32, 33, 34, 35, 36, 37, 38])
def test_tiny_full_oracle_every_plan(plan_id):
    res = Hh.run_request(I.config_tiny(), plan_id=plan_id)
    assert res["pairs"] == res["info"]["nnz_blocks"] * 64 * 64


@pytest.mark.parametrize("plan_id", [-1, 0, 1, 2, 4, 6, 7, 8, 10, 12, 14, 16, 18, 20, 22, 24, 25, 26, 29, 30, 31])
def test_mid_full_oracle(plan_id):
    """-1 is the configuration bench.py times (the plan the shipped table selects); every row is compared."""
    Hh.run_request(I.config_mid(), plan_id=plan_id)


def test_hunyuan_shaped_sampled_oracle():
    req = I.config_hunyuan()
    # 64 seeded query blocks per head; structure (coverage, CSR, items) on three heads to bound host time
    Hh.run_request(req, plan_id=-1, sel=_sample(req, 64), heads=[0, 11, 23])


@pytest.mark.parametrize("plan_id", [-1, 0, 1, 10, 14, 18, 22, 23, 25])
def test_stress_a_coarsened(plan_id):
    req = I.config_stress_a()
    res = Hh.run_request(req, plan_id=plan_id, sel=_sample(req, 64), heads=[0, 15])
    if bsa.catalog()[res["info"]["plan"]["plan_id"]]["kernel"] != 5:
        assert res["info"]["map_q"] == 1  # Coarsened along Q: 8 logical rows of 16 per 128-row tile


@pytest.mark.parametrize("plan_id", [34, 35, 37])
def test_stress_a_on_16_row_tiles(plan_id):
    """The same request on the row-block kernel: every 16-row logical block is its own physical tile (Direct along Q,
    Direct or Refined along KV), so the plan covers exactly the active pairs."""
    req = I.config_stress_a()
    res = Hh.run_request(req, plan_id=plan_id, sel=_sample(req, 64), heads=[3])
    inf = res["info"]
    assert inf["map_q"] == 0 and inf["plan"]["T_Q"] == 16 and inf["covered_pairs"] == res_pairs(req)


def res_pairs(req):
    return oracle.active_pairs(req.mask, req.B_Q, req.B_KV, req.N, req.n_kv)


@pytest.mark.parametrize("plan_id", [-1, 0, 1, 10, 11, 14, 15, 18, 19, 22, 23, 25])
def test_stress_b_refined(plan_id):
    req = I.config_stress_b()
    res = Hh.run_request(req, plan_id=plan_id, sel=_sample(req, 64))
    # B = (256,256): Refined along KV always; along Q Refined for 128-row tiles, Direct for 256-row tiles
    assert res["info"]["map_kv"] == 2 and res["info"]["map_q"] == (2 if res["info"]["plan"]["T_Q"] == 128 else 0)


@pytest.mark.parametrize("r,B,rho", [(0, (32, 32), 0.03), (1, (64, 128), 0.10), (2, (128, 64), 0.30),
                                     (3, (256, 256), 0.60), (4, (128, 128), 0.03), (5, (32, 32), 0.60)])
def test_sweep_requests_ragged_n(r, B, rho):
    """Dynamic-request sweep shapes (N = 75600 is not a multiple of any block size): 64 seeded query blocks per head
    against the oracle.  On the requests of 30 % density and more a seeded subset of the rows of every sampled block
    (every 4th row; rows are independent) bounds the oracle's time.  6 heads keep the host-side mask generation short;
    the full 24 heads are in the next test."""
    req = I.config_sweep(r, H=6, B=B, rho=rho)
    Hh.run_request(req, plan_id=-1, sel=_sample(req, 64), row_step=4 if rho >= 0.3 else 1, heads=[0, 5])


@pytest.mark.parametrize("plan_id,rho", [(35, 0.03), (38, 0.10), (36, 0.03)])
def test_sweep_32x32_request_on_16_row_tiles(plan_id, rho):
    """A (32,32) sweep request (d = 128, ragged N) on the row-block kernel: two 16-row tiles per logical row block
    (Refined along Q), 32- or 16-key tiles, no pair outside E(M) computed."""
    req = I.config_sweep(1, H=6, B=(32, 32), rho=rho)
    res = Hh.run_request(req, plan_id=plan_id, sel=_sample(req, 64), heads=[5])
    inf = res["info"]
    # whole 16 x T_KV tiles are counted, so only the ragged last block row and column add to the active pairs
    assert inf["map_q"] == 2 and res_pairs(req) <= inf["covered_pairs"] <= inf["nnz_blocks"] * 32 * 32
    assert inf["covered_pairs"] < 1.001 * res_pairs(req)


@pytest.mark.parametrize("r,B,rho,row_step", [(7, (32, 32), 0.30, 4), (8, (128, 128), 0.10, 1)])
def test_sweep_requests_at_all_24_heads(r, B, rho, row_step):
    """Two sweep requests at their stated size (24 heads x 75600 tokens, d = 128), 64 seeded query blocks per head.
    The (32,32) one at 30 % has the planner's largest structures (a 134 MB mask, 37 million active blocks and as many
    tile-list entries, within a factor of 60 of the planner's 32-bit tile-index capacity); plan coverage is checked bit for bit on
    two heads, statistics and block-CSR on all."""
    req = I.config_sweep(r, H=24, B=B, rho=rho)
    res = Hh.run_request(req, plan_id=-1, sel=_sample(req, 64), row_step=row_step, heads=[0, 23])
    assert res["info"]["lut_hit"] == 1


# ---------------------------------------------------------------- small geometries spanning tiles + ragged tails
@pytest.mark.parametrize("B_Q,B_KV,N,d,plan_id", [
    (16, 16, 1000, 64, 0), (16, 16, 1000, 64, 1), (32, 64, 777, 128, 0), (64, 32, 1300, 128, 1),
    (128, 256, 2100, 64, 0), (256, 128, 2100, 128, 1), (256, 16, 900, 64, 3), (16, 256, 900, 128, 2),
    (64, 64, 130, 64, 0), (128, 128, 127, 128, 0), (128, 128, 1, 64, 1),
    (16, 16, 1000, 64, 10), (32, 64, 777, 128, 11), (64, 32, 1300, 128, 10), (128, 256, 2100, 64, 11),
    (256, 128, 2100, 128, 10), (256, 16, 900, 64, 12), (16, 256, 900, 128, 12), (128, 128, 127, 128, 10),
    (128, 128, 129, 64, 10), (64, 64, 300, 128, 13),
    (16, 16, 1000, 64, 14), (32, 64, 777, 128, 15), (64, 32, 1300, 128, 14), (128, 256, 2100, 64, 15),
    (256, 128, 2100, 128, 14), (256, 16, 900, 64, 16), (16, 256, 900, 128, 16), (128, 128, 127, 128, 17),
    (16, 16, 1000, 64, 18), (32, 64, 777, 128, 19), (64, 32, 1300, 128, 18), (128, 256, 2100, 64, 19),
    (256, 128, 2100, 128, 18), (256, 16, 900, 64, 20), (16, 256, 900, 128, 20), (128, 128, 127, 128, 21),
    (16, 16, 1000, 64, 22), (32, 64, 777, 128, 23), (64, 32, 1300, 128, 22), (128, 256, 2100, 64, 23),
    (256, 128, 2100, 128, 22), (256, 16, 900, 64, 24), (16, 256, 900, 128, 24), (128, 128, 127, 128, 25),
    (64, 64, 130, 64, 22), (128, 128, 1, 64, 23), (128, 128, 129, 128, 22), (32, 32, 3000, 64, 25),
    (16, 16, 1000, 64, 36), (32, 64, 777, 128, 35), (64, 32, 1300, 128, 35), (16, 256, 900, 128, 38), (16, 64, 1000, 64, 34),
    (32, 32, 3000, 64, 35), (64, 128, 2100, 64, 37), (64, 64, 130, 64, 34), (16, 16, 1, 128, 36), (32, 256, 1111, 64, 34),
])
def test_geometries_with_ragged_tail(B_Q, B_KV, N, d, plan_id):
    H = 3
    M = I.random_mask(B_Q * 131 + B_KV + N, H, I.cdiv(N, B_Q), I.cdiv(N, B_KV), 0.35, diag=True, empty_rows=0.15)
    req = I.Request("geom", H, N, d, B_Q, B_KV, M, qkv_seed=N + d)
    Hh.run_request(req, plan_id=plan_id)


# ---------------------------------------------------------------- degenerate masks
@pytest.mark.parametrize("kind", ["empty", "full", "one_block", "empty_head"])
def test_degenerate_masks(kind):
    H, N, d, B = 2, 512, 64, 64
    nb = N // B
    M = np.zeros((H, nb, nb), np.uint8)
    if kind == "full":
        M[:] = 1
    elif kind == "one_block":
        M[1, 3, 5] = 1
    elif kind == "empty_head":
        M[0] = I.random_mask(1, 1, nb, nb, 0.5)[0]
    req = I.Request(kind, H, N, d, B, B, M, qkv_seed=3)
    for plan_id in (0, 3, 10, 12, 14, 16, 18, 20, 22, 24, 34, 36):
        Hh.run_request(req, plan_id=plan_id)


# ---------------------------------------------------------------- closed forms on the GPU path
@pytest.mark.parametrize("B_Q,B_KV,N,d,plan_id", [(16, 64, 1000, 64, 0), (32, 32, 700, 128, 1), (256, 256, 1100, 128, 9),
                                                  (16, 64, 1000, 64, 10), (64, 32, 700, 128, 11), (256, 256, 1100, 128, 12),
                                                  (16, 64, 1000, 64, 14), (64, 32, 700, 128, 15), (256, 256, 1100, 128, 16),
                                                  (16, 64, 1000, 64, 18), (64, 32, 700, 128, 19), (256, 256, 1100, 128, 20),
                                                  (16, 64, 1000, 64, 22), (64, 32, 700, 128, 23), (256, 256, 1100, 128, 24),
                                                  (16, 64, 1000, 64, 34), (64, 32, 700, 128, 35), (32, 16, 900, 128, 36)])
def test_zero_keys_give_log_count_and_mean_value(B_Q, B_KV, N, d, plan_id):
    """K = 0: every score is 0, so LSE = ln(#reachable keys) exactly and O = mean of reachable V.
    Catches any off-by-one in ragged-edge or membership masking (one key off moves LSE by ~1/count)."""
    H = 2
    M = I.random_mask(5, H, I.cdiv(N, B_Q), I.cdiv(N, B_KV), 0.3, diag=True, empty_rows=0.1)
    q, k, v = I.make_qkv(1, H, N, d)
    mask = torch.from_numpy(M).cuda()
    with bsa.plan_create(mask, B_Q, B_KV, N, H, d, plan_id=plan_id) as plan:
        O, LSE = plan.forward(q.cuda(), torch.zeros_like(k).cuda(), v.cuda())
        torch.cuda.synchronize()
    ck = np.minimum(B_KV, N - np.arange(M.shape[2]) * B_KV)
    cnt = np.repeat((M * ck[None, None, :]).sum(axis=2), B_Q, axis=1)[:, :N]
    LSE = LSE.cpu().numpy()
    nz = cnt > 0
    assert np.array_equal(np.isneginf(LSE), ~nz)
    np.testing.assert_allclose(LSE[nz], np.log(cnt[nz]), atol=2e-6, rtol=0)
    # O = mean of the reachable values (bf16 output rounding only)
    E = np.repeat(np.repeat(M[0] != 0, B_Q, axis=0), B_KV, axis=1)[:N, :N]
    v64 = v[0].double().numpy()
    mean = (E @ v64) / np.maximum(cnt[0], 1)[:, None]
    np.testing.assert_allclose(O[0].float().cpu().numpy()[nz[0]], mean[nz[0]], atol=4e-3, rtol=0)


def test_constant_values_come_back():
    H, N, d = 2, 900, 128
    M = I.random_mask(8, H, I.cdiv(N, 64), I.cdiv(N, 32), 0.4, diag=True)
    q, k, v = I.make_qkv(2, H, N, d)
    vc = torch.full_like(v, 0.75)
    with bsa.plan_create(torch.from_numpy(M).cuda(), 64, 32, N, H, d, plan_id=0) as plan:
        O, _ = plan.forward(q.cuda(), k.cuda(), vc.cuda())
        torch.cuda.synchronize()
    assert torch.allclose(O.float(), torch.full_like(O.float(), 0.75), atol=4e-3)


@pytest.mark.parametrize("plan_id", [1, 18, 22, 23, 24])
def test_sharp_scores_stay_within_tolerance(plan_id):
    # 4x larger scores: a much peakier softmax, the reference maximum keeps moving and the running output is
    # rescaled often (in the ping-pong kernel the reference is handed from one warpgroup to the other every tile)
    req = I.config_tiny(seed=21)
    q, k, v = req.qkv()
    res = Hh.run_request(req, plan_id=plan_id, qkv=((q * 2).to(torch.bfloat16), (k * 2).to(torch.bfloat16), v),
                         guards=False)
    assert res["lse_max"] < 2e-4


@pytest.mark.parametrize("plan_id", [18, 22])
def test_growing_scores_force_a_rescale_at_every_tile(plan_id):
    """Keys sorted by increasing magnitude along the sequence: every later tile raises the row maximum by more
    than the rescale threshold, so the reference moves (and O is rescaled) tile after tile."""
    H, N, d, B = 1, 1024, 128, 128
    q, k, v = I.make_qkv(77, H, N, d)
    ramp = torch.linspace(0.2, 6.0, N).view(1, N, 1)
    k = (k * ramp).to(torch.bfloat16)
    M = np.ones((H, N // B, N // B), np.uint8)
    req = I.Request("ramp", H, N, d, B, B, M, qkv_seed=0)
    res = Hh.run_request(req, plan_id=plan_id, qkv=(q, k, v), guards=False)
    assert res["lse_max"] < 5e-4


@pytest.mark.parametrize("name,plan_id", [("stress_b", 22), ("stress_b", 23), ("stress_b", 18), ("mid", 22), ("mid", 24),
                                          ("stress_a", 23), ("tiny", 27), ("stress_a", 34), ("tiny", 36)])
def test_repeated_runs_are_bitwise_identical(name, plan_id):
    """No atomics and a fixed accumulation order: six forwards of one plan give the same bits.  Long work items
    (Stress-B has about a hundred tiles per item) give a timing-dependent hand-off the most chances to show."""
    req = I.CONFIGS[name]()
    mask, q, k, v, _ = Hh.to_dev(req, None)
    with bsa.plan_create(mask, req.B_Q, req.B_KV, req.N, req.H, req.d, plan_id=plan_id) as plan:
        O0, L0 = plan.forward(q, k, v)
        torch.cuda.synchronize()
        O0, L0 = O0.clone(), L0.clone()
        for _ in range(5):
            O, L = plan.forward(q, k, v)
            torch.cuda.synchronize()
            assert torch.equal(O, O0) and torch.equal(L, L0)
        assert plan.info()["device_status"] == 0


@pytest.mark.parametrize("d,plan_id", [(64, 22), (64, 23), (128, 22), (64, 18), (128, 25)])
def test_many_single_tile_items(d, plan_id):
    """Block-diagonal mask: every work item has one tile (two with 64-wide tiles), so the producers run several
    items ahead of the MMA issuers and the queue of pending Q tiles fills up (deep rings at d = 64)."""
    H, B, nb = 2, 128, 300
    N = B * nb - 37  # ragged last block
    M = np.zeros((H, nb, nb), np.uint8)
    M[:, np.arange(nb), np.arange(nb)] = 1
    M[1, 5, :] = 0  # one empty row among them
    req = I.Request("diag", H, N, d, B, B, M, qkv_seed=5)
    Hh.run_request(req, plan_id=plan_id)


# ---------------------------------------------------------------- boundary behaviour
def test_invalid_arguments_never_touch_the_gpu():
    import ctypes
    L = bsa.lib()
    h = ctypes.c_void_p()
    m = torch.zeros((1, 2, 2), dtype=torch.uint8, device="cuda")
    assert L.bsa_plan_create(None, 64, 64, 128, 1, 64, ctypes.byref(h)) == 1
    assert L.bsa_plan_create(m.data_ptr(), 64, 64, 0, 1, 64, ctypes.byref(h)) == 1
    assert L.bsa_plan_create(m.data_ptr(), 48, 64, 128, 1, 64, ctypes.byref(h)) == 2
    assert L.bsa_plan_create(m.data_ptr(), 64, 64, 128, 1, 96, ctypes.byref(h)) == 2
    assert L.bsa_plan_create(m.data_ptr(), 64, 512, 128, 1, 64, ctypes.byref(h)) == 2
    with pytest.raises(bsa.BsaError) as e:
        bsa.plan_create(m, 64, 64, 128, 1, 64, plan_id=2, max_workspace_bytes=1024)  # workspace too small
    assert e.value.status == 3
    with bsa.plan_create(m, 64, 64, 128, 1, 64) as plan:
        q = torch.zeros((1, 128, 64), dtype=torch.bfloat16, device="cuda")
        assert L.bsa_forward(plan._h, q.data_ptr() + 2, q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(), None) == 1
        assert L.bsa_forward(plan._h, None, q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(), None) == 1


def test_request_from_host_buffers_matches_device_path():
    req = I.config_tiny(seed=4, N=1536)
    q, k, v = req.qkv()
    O = torch.empty_like(q)
    LSE = torch.empty((req.H, req.N), dtype=torch.float32)
    inf = bsa.request_host(req.mask, req.B_Q, req.B_KV, req.N, req.H, req.d, q, k, v, O, LSE)
    assert inf["device_status"] == 0
    Hh.compare_with_oracle(req, O, LSE, (q, k, v))


def test_pipelined_request_from_pinned_host_buffers():
    """The bench's end-to-end path on its own workload: bsa_request_host cuts Mid's 8 heads into 3 groups and
    pipelines copies in, planning + forward, and copies out.  Outputs against the oracle on sampled query blocks of
    every head; the aggregated info equals the whole mask's statistics and the sums over heads."""
    req = I.config_mid()
    q, k, v = req.qkv()
    qp, kp, vp = (t.pin_memory() for t in (q, k, v))
    O = torch.empty_like(q).pin_memory()
    LSE = torch.empty((req.H, req.N), dtype=torch.float32).pin_memory()
    mask = torch.from_numpy(req.mask).pin_memory()
    O.fill_(float("nan"))
    LSE.fill_(float("nan"))
    inf = bsa.request_host(mask, req.B_Q, req.B_KV, req.N, req.H, req.d, qp, kp, vp, O, LSE)
    assert inf["device_status"] == 0 and inf["heads"] == req.H
    Hh.compare_with_oracle(req, O, LSE, (q, k, v), sel=_sample(req, 16))
    with bsa.plan_create(torch.from_numpy(req.mask).cuda(), req.B_Q, req.B_KV, req.N, req.H, req.d) as whole:
        w = whole.info()
    for key in ("nnz_blocks", "blocks_in_runs", "max_row_nnz", "ntiles", "nitems", "covered_pairs"):
        assert inf[key] == w[key], key
    for key in ("density", "run_coverage", "skew"):
        assert abs(inf[key] - w[key]) < 1e-9, key


def test_dense_coarsened_mask_takes_the_bit_plane_tile_map():
    """From 1536 active blocks per tile row on, a Coarsened mask with a small membership word is mapped by the
    bit-plane kernel (one bitmap per membership bit instead of one word per tile column): (32,32) blocks at 50 %
    density, N = 32768, on 128x64 tiles has 2048 per tile row.  Tile lists and membership words against the oracle bit
    for bit, outputs on sampled query blocks; the same plan on a sparse mask of the same shape takes the other kernel."""
    for p_active in (0.5, 0.05):
        req = I.config_tiny(seed=41, H=2, N=32768, d=128, B=32, p=p_active)
        pid = next(i for i, c in enumerate(bsa.catalog()) if c["name"] == "q128k64_pp_gb")
        Hh.run_request(req, plan_id=pid, sel=_sample(req, 2), guards=False)


def test_host_request_with_tapered_head_groups():
    """With more than 32 MB of Q, K, V per head a group may be a single head, and bsa_request_host then tapers the
    groups towards the end (12 heads: 3 2 2 2 2 1) so that little work is left after the last input byte.  Every head
    lands in the right place: outputs against the oracle on sampled query blocks of every head, no row left unwritten,
    and the aggregated counts equal those of one plan over the whole mask."""
    req = I.config_tiny(seed=31, H=12, N=49152, d=128, B=128, p=0.01)   # 37.7 MB of Q, K, V per head
    q, k, v = req.qkv()
    qp, kp, vp = (t.pin_memory() for t in (q, k, v))
    O = torch.empty_like(q).pin_memory()
    LSE = torch.empty((req.H, req.N), dtype=torch.float32).pin_memory()
    O.fill_(float("nan"))
    LSE.fill_(float("nan"))
    inf = bsa.request_host(torch.from_numpy(req.mask).pin_memory(), req.B_Q, req.B_KV, req.N, req.H, req.d, qp, kp, vp, O, LSE)
    assert inf["device_status"] == 0 and inf["heads"] == req.H
    assert not torch.isnan(O.float()).any() and not torch.isnan(LSE).any()
    Hh.compare_with_oracle(req, O, LSE, (q, k, v), sel=_sample(req, 4))
    with bsa.plan_create(torch.from_numpy(req.mask).cuda(), req.B_Q, req.B_KV, req.N, req.H, req.d) as whole:
        w = whole.info()
    for key in ("nnz_blocks", "blocks_in_runs", "max_row_nnz", "ntiles", "nitems", "covered_pairs"):
        assert inf[key] == w[key], key


@pytest.mark.parametrize("plan_id", [22, 27])
def test_forward_replays_from_a_cuda_graph(plan_id):
    """bsa_forward only launches kernels (no allocation, no synchronisation): it can be captured into a CUDA graph
    and replayed, with and without Split-K, and the replay gives the bits of the direct call."""
    req = I.config_tiny()
    mask, q, k, v, _ = Hh.to_dev(req, None)
    with bsa.plan_create(mask, req.B_Q, req.B_KV, req.N, req.H, req.d, plan_id=plan_id) as plan:
        O0, L0 = plan.forward(q, k, v)  # also sets the kernels' shared-memory attributes before the capture
        torch.cuda.synchronize()
        O = torch.zeros_like(O0)
        L = torch.zeros_like(L0)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                plan.forward(q, k, v, O, L, stream=side)
        for _ in range(3):
            O.zero_()
            L.zero_()
            graph.replay()
            torch.cuda.synchronize()
            assert torch.equal(O, O0) and torch.equal(L, L0)
        assert plan.info()["device_status"] == 0


@pytest.mark.parametrize("B_Q,B_KV,N,d,plan_id", [(16, 16, 1000, 64, 22), (32, 64, 4100, 128, 23), (128, 128, 16384, 128, -1),
                                                  (16, 32, 40000, 64, 25), (256, 16, 9000, 128, 1), (64, 64, 130, 64, 27)])
def test_bit_packed_mask_gives_the_same_plan_and_output(B_Q, B_KV, N, d, plan_id):
    """bsa_plan_create_packed reads the mask as bits: statistics, block-CSR, tiles, work items and the forward's output
    are those of the byte-mask plan, bit for bit (row lengths that are not multiples of 8 or 32 blocks included)."""
    H = 3
    M = I.random_mask(11, H, I.cdiv(N, B_Q), I.cdiv(N, B_KV), 0.3)
    M[1, 2, :] = 0
    req = I.Request("packed", H, N, d, B_Q, B_KV, M, qkv_seed=9)
    mask, q, k, v, _ = Hh.to_dev(req, None)
    bits, stride = bsa.pack_mask(mask)
    with bsa.plan_create(mask, B_Q, B_KV, N, H, d, plan_id=plan_id) as pa, \
            bsa.plan_create_packed(bits, stride, B_Q, B_KV, N, H, d, plan_id=plan_id) as pb:
        ia, ib = pa.info(), pb.info()
        for key in ("nnz_blocks", "blocks_in_runs", "max_row_nnz", "density", "run_coverage", "skew", "ntiles", "nitems"):
            assert ia[key] == ib[key], key
        assert ia["plan"]["plan_id"] == ib["plan"]["plan_id"]
        for x, y in zip(pa.export_csr(), pb.export_csr()):
            assert np.array_equal(x, y)
        for h in range(H):
            for x, y in zip(pa.export_tiles(h), pb.export_tiles(h)):
                assert np.array_equal(x, y)
        assert np.array_equal(pa.export_items(), pb.export_items())
        Oa, La = pa.forward(q, k, v)
        Ob, Lb = pb.forward(q, k, v)
        torch.cuda.synchronize()
        assert torch.equal(Oa, Ob) and torch.equal(La, Lb)


# ---------------------------------------------------------------- N_q != N_kv (Section 2.1: Q is N_q x d, K and V are N_kv x d)
@pytest.mark.parametrize("B_Q,B_KV,N_q,N_kv,d,plan_id", [
    (64, 64, 1000, 3000, 64, -1), (64, 64, 1000, 3000, 64, 22), (128, 128, 2100, 700, 128, -1),
    (16, 32, 900, 2500, 64, 25), (32, 16, 2500, 900, 128, 0), (128, 64, 130, 4000, 128, 2),
    (256, 128, 1500, 520, 64, 1), (64, 256, 600, 2050, 128, 10), (128, 128, 4096, 128, 128, 23),
    (16, 16, 300, 1111, 64, 14), (64, 64, 1000, 3000, 128, 24), (32, 32, 3000, 1000, 64, 18),
    (128, 128, 1, 777, 128, -1), (64, 64, 777, 1, 64, -1), (16, 64, 900, 2500, 64, 34), (32, 32, 2500, 900, 128, 35),
    (64, 16, 777, 1, 64, 36)])
def test_rectangular_requests_match_the_oracle(B_Q, B_KV, N_q, N_kv, d, plan_id):
    """More (or fewer) key tokens than query tokens: ragged last blocks on both sides, every kernel family,
    Direct / Coarsened / Refined mappings, Split-K plans; all rows compared, tile plan == E(M)."""
    H = 3
    M = I.random_mask(41, H, I.cdiv(N_q, B_Q), I.cdiv(N_kv, B_KV), 0.35, empty_rows=0.1)
    req = I.Request("rect", H, N_q, d, B_Q, B_KV, M, qkv_seed=17, N_kv=N_kv)
    # the stated tolerances apply; the tighter regression guards assume hundreds of keys per row, and here a row may
    # see a handful (one probability near 1 rounded to bf16 moves O by up to 2^-9 max|v|)
    res = Hh.run_request(req, plan_id=plan_id, guards=False)
    inf = res["info"]
    assert (inf["N"], inf["N_kv"]) == (N_q, N_kv)
    assert (inf["nQb"], inf["nKb"]) == (I.cdiv(N_q, B_Q), I.cdiv(N_kv, B_KV))
    assert res["pairs"] == oracle.active_pairs(M, B_Q, B_KV, N_q, N_kv)


def test_rectangular_request_from_host_buffers_packed_mask_and_cache():
    B_Q, B_KV, N_q, N_kv, d, H = 64, 128, 1500, 5000, 128, 2
    M = I.random_mask(43, H, I.cdiv(N_q, B_Q), I.cdiv(N_kv, B_KV), 0.3)
    req = I.Request("rect_host", H, N_q, d, B_Q, B_KV, M, qkv_seed=19, N_kv=N_kv)
    mask, q, k, v, qkv_cpu = Hh.to_dev(req)
    with bsa.plan_create(mask, B_Q, B_KV, N_q, H, d, N_kv=N_kv) as plan:
        O, LSE = plan.forward(q, k, v)
        torch.cuda.synchronize()
        Hh.compare_with_oracle(req, O, LSE, qkv_cpu)
    # host buffers
    Oh = torch.empty_like(qkv_cpu[0])
    Lh = torch.empty((H, N_q), dtype=torch.float32)
    bsa.request_host(req.mask, B_Q, B_KV, N_q, H, d, *qkv_cpu, Oh, Lh, N_kv=N_kv)
    assert torch.equal(Oh, O.cpu()) and torch.equal(Lh, LSE.cpu())
    # bit-packed mask and the plan cache (N_kv is part of its key)
    bits, stride = bsa.pack_mask(mask)
    with bsa.plan_create_packed(bits, stride, B_Q, B_KV, N_q, H, d, N_kv=N_kv) as pb:
        Ob, Lb = pb.forward(q, k, v)
        torch.cuda.synchronize()
        assert torch.equal(Ob, O) and torch.equal(Lb, LSE)
    cache = bsa.PlanCache(4)
    p0, h0 = cache.get(mask, B_Q, B_KV, N_q, H, d, N_kv=N_kv)
    p1, h1 = cache.get(mask, B_Q, B_KV, N_q, H, d, N_kv=N_kv)
    assert (h0, h1) == (False, True)
    Oc, Lc = p1.forward(q, k, v)
    torch.cuda.synchronize()
    assert torch.equal(Oc, O) and torch.equal(Lc, LSE)
    p0.destroy(); p1.destroy()
    # the same mask array read with another N_kv that gives the same block grid is another request
    p2, h2 = cache.get(mask, B_Q, B_KV, N_q, H, d, N_kv=N_kv - 1)
    assert not h2
    p2.destroy()
    cache.destroy()


# ---------------------------------------------------------------- fp16 tensors (request property x, Section 4.4)
@pytest.mark.parametrize("B_Q,B_KV,N,N_kv,d,plan_id", [
    (128, 128, 4096, 0, 128, -1), (64, 64, 3000, 0, 64, -1), (128, 128, 2100, 0, 128, 23), (16, 32, 1500, 0, 64, 25),
    (128, 64, 2000, 0, 128, 26), (64, 64, 2048, 0, 64, 24), (32, 32, 1000, 2500, 128, 29), (128, 128, 4096, 0, 64, 33),
    (128, 128, 2100, 0, 128, 0), (64, 32, 1300, 0, 64, 3), (16, 64, 1500, 0, 128, 18), (256, 256, 1500, 0, 64, 19),
    (16, 64, 1000, 0, 64, 34), (32, 32, 900, 1700, 128, 35), (64, 16, 700, 0, 64, 36),
    (128, 128, 1500, 0, 256, -1), (32, 64, 900, 0, 256, 3)])
def test_half_precision_requests_match_the_oracle(B_Q, B_KV, N, N_kv, d, plan_id):
    """Q, K, V, O in IEEE half: the fp16 instantiations of the ping-pong kernel (both head dims and tile widths,
    Direct / Coarsened / Refined mappings, Split-K with the merge kernel's half output), of the single-tile kernels
    (one and two issuers, Split-K, d = 256) and of the row-block kernel, all rows against the oracle reading the same
    half bit patterns."""
    H = 3
    M = I.random_mask(61, H, I.cdiv(N, B_Q), I.cdiv(N_kv or N, B_KV), 0.35, empty_rows=0.1)
    req = I.Request("half", H, N, d, B_Q, B_KV, M, qkv_seed=23, N_kv=N_kv, dtype="fp16")
    res = Hh.run_request(req, plan_id=plan_id)
    assert res["info"]["dtype"] == 1
    assert bsa.catalog()[res["info"]["plan"]["plan_id"]]["kernel"] in (0, 3, 4, 5)


def test_half_precision_mid_and_ineligible_plans():
    """The Mid shape in half; plans of the paired and column-split kernels are not eligible for a half request (forced:
    no eligible plan; looked up: the ranking falls through to the next plan that is)."""
    req = I.config_mid()
    req.dtype = "fp16"
    Hh.run_request(req, plan_id=-1, sel=_sample(req, 16))
    mask, q, k, v, _ = Hh.to_dev(I.config_tiny())
    t = I.config_tiny()
    with pytest.raises(bsa.BsaError) as e:
        bsa.plan_create(mask, t.B_Q, t.B_KV, t.N, t.H, t.d, plan_id=14, dtype="fp16")
    assert e.value.status == 3
    # the same bits through a bf16 plan and a half plan differ: the plan's dtype is what the kernel reads
    th = I.config_tiny()
    th.dtype = "fp16"
    _, qh, kh, vh, _ = Hh.to_dev(th)
    with bsa.plan_create(mask, t.B_Q, t.B_KV, t.N, t.H, t.d, dtype="fp16") as ph, \
            bsa.plan_create(mask, t.B_Q, t.B_KV, t.N, t.H, t.d, plan_id=ph.info()["plan"]["plan_id"]) as pb:
        Oh, _ = ph.forward(qh, kh, vh)
        Ob, _ = pb.forward(qh.view(torch.bfloat16), kh.view(torch.bfloat16), vh.view(torch.bfloat16))
        torch.cuda.synchronize()
        assert not torch.equal(Oh.view(torch.int16), Ob.view(torch.int16))


# ---------------------------------------------------------------- head dimension 256 (a tensor property of the request)
@pytest.mark.parametrize("B_Q,B_KV,N,N_kv,plan_id", [(128, 128, 2100, 0, -1), (64, 64, 1000, 0, 19), (16, 32, 900, 1500, 1),
                                                      (256, 256, 1500, 0, 3), (128, 64, 3000, 0, 5), (32, 16, 700, 0, 9)])
def test_head_dim_256_matches_the_oracle(B_Q, B_KV, N, N_kv, plan_id):
    """d = 256: the output accumulator takes half of tensor memory, so the request is served by the single-tile kernels
    (P in place over S) with 64-key tiles, Split-K included; every other plan is ineligible and the base plan of the
    key is one of those kernels.  All rows against the oracle, tile plan == E(M)."""
    H, d = 2, 256
    M = I.random_mask(91, H, I.cdiv(N, B_Q), I.cdiv(N_kv or N, B_KV), 0.35, diag=True, empty_rows=0.1)
    req = I.Request("d256", H, N, d, B_Q, B_KV, M, qkv_seed=37, N_kv=N_kv)
    res = Hh.run_request(req, plan_id=plan_id, guards=False)
    cat = bsa.catalog()[res["info"]["plan"]["plan_id"]]
    assert cat["kernel"] in (0, 3) and cat["T_KV"] == 64 and res["info"]["d"] == 256
    mask = torch.from_numpy(M).cuda()
    for bad in (22, 18, 10, 14, 36):     # ping-pong, 128-key tiles, paired, column-split, row-block
        with pytest.raises(bsa.BsaError) as e:
            bsa.plan_create(mask, B_Q, B_KV, N, H, d, plan_id=bad, N_kv=N_kv)
        assert e.value.status == 3


# ---------------------------------------------------------------- token-major layout [N, heads, d]
@pytest.mark.parametrize("B_Q,B_KV,N,N_kv,d,dtype", [(64, 64, 2048, 0, 64, "bf16"), (128, 128, 3000, 0, 128, "bf16"),
                                                      (32, 64, 1500, 2600, 128, "bf16"), (128, 128, 2500, 0, 128, "fp16")])
def test_token_major_layout_gives_the_same_output(B_Q, B_KV, N, N_kv, d, dtype):
    """Q, K, V, O stored [N, heads, d] (the layout is a tensor property of the request): one plan per kernel family
    and a Split-K plan give, permuted back, the bits of the head-major run; the first is also compared with the oracle."""
    H = 3
    M = I.random_mask(81, H, I.cdiv(N, B_Q), I.cdiv(N_kv or N, B_KV), 0.3, empty_rows=0.1)
    req = I.Request("nhd", H, N, d, B_Q, B_KV, M, qkv_seed=31, N_kv=N_kv, dtype=dtype)
    mask, q, k, v, qkv_cpu = Hh.to_dev(req)
    qt, kt, vt = (t.permute(1, 0, 2).contiguous() for t in (q, k, v))
    cat = bsa.catalog()
    plans = []
    for kern in (4, 0, 1, 2, 3, 5):
        ids = [c["plan_id"] for c in cat if c["kernel"] == kern and c["split_pmax"] == 1 and
               bsa.plan_eligible(c["plan_id"], B_Q, B_KV, N, H, d, N_kv=N_kv, dtype=dtype)]
        plans += ids[:1]
    plans += [c["plan_id"] for c in cat if c["split_pmax"] > 1 and
              bsa.plan_eligible(c["plan_id"], B_Q, B_KV, N, H, d, N_kv=N_kv, dtype=dtype)][:1]
    assert len(plans) >= (6 if dtype == "bf16" else 2)
    for n, pid in enumerate(plans):
        with bsa.plan_create(mask, B_Q, B_KV, N, H, d, plan_id=pid, N_kv=N_kv, dtype=dtype) as pa, \
                bsa.plan_create(mask, B_Q, B_KV, N, H, d, plan_id=pid, N_kv=N_kv, dtype=dtype, layout="nhd") as pb:
            assert pb.info()["layout"] == 1 and pa.info()["layout"] == 0
            Oa, La = pa.forward(q, k, v)
            Ob, Lb = pb.forward(qt, kt, vt)
            torch.cuda.synchronize()
            assert Ob.shape == (N, H, d) and Lb.shape == (H, N)
            assert torch.equal(Ob.permute(1, 0, 2), Oa) and torch.equal(La, Lb), pid
            if n == 0:
                Hh.compare_with_oracle(req, Ob.permute(1, 0, 2).contiguous(), Lb, qkv_cpu)


@pytest.mark.parametrize("B_Q,B_KV,N,N_kv,d,dtype,plan_id", [(64, 64, 1000, 0, 64, "bf16", -1), (128, 128, 1500, 2100, 128, "bf16", 22),
                                                              (32, 64, 900, 0, 128, "fp16", -1), (16, 64, 700, 0, 64, "bf16", 34)])
def test_batched_token_major_request(B_Q, B_KV, N, N_kv, d, dtype, plan_id):
    """Explicit batch (a request dimension): tensors stored [batch, N, heads, d] with `heads` counting batch x heads
    problems.  The output equals, problem by problem, the head-major run of the folded request (bit for bit) and the
    oracle; the info sums the batch elements; exports and the plan cache refuse such a plan; with the head-major
    layout the batch option changes nothing."""
    Bt, Hb = 3, 2
    H = Bt * Hb
    M = I.random_mask(97, H, I.cdiv(N, B_Q), I.cdiv(N_kv or N, B_KV), 0.3, empty_rows=0.1)
    req = I.Request("batched", H, N, d, B_Q, B_KV, M, qkv_seed=41, N_kv=N_kv, dtype=dtype)
    mask, q, k, v, qkv_cpu = Hh.to_dev(req)
    args = (B_Q, B_KV, N, H, d)
    kw = dict(plan_id=plan_id, N_kv=N_kv, dtype=dtype)

    def to_bnhd(t):   # [B*Hb, n, d] -> [B, n, Hb, d]
        return t.view(Bt, Hb, t.shape[1], d).permute(0, 2, 1, 3).contiguous()

    with bsa.plan_create(mask, *args, **kw) as plain, bsa.plan_create(mask, *args, layout="nhd", batch=Bt, **kw) as batched, \
            bsa.plan_create(mask, *args, batch=Bt, **kw) as folded:
        O, L = plain.forward(q, k, v)
        Ob, Lb = batched.forward(to_bnhd(q), to_bnhd(k), to_bnhd(v))
        Of, Lf = folded.forward(q, k, v)
        torch.cuda.synchronize()
        assert Ob.shape == (Bt, N, Hb, d) and Lb.shape == (H, N)
        if plan_id >= 0:   # the same catalog plan everywhere: the same bits (a lookup may choose per batch element)
            assert torch.equal(Ob.permute(0, 2, 1, 3).reshape(H, N, d), O) and torch.equal(Lb, L)
        assert torch.equal(Of, O) and torch.equal(Lf, L)
        Hh.compare_with_oracle(req, Ob.permute(0, 2, 1, 3).reshape(H, N, d).contiguous(), Lb, qkv_cpu, guards=False)
        ia, ib = plain.info(), batched.info()
        for key in ("heads", "nnz_blocks", "blocks_in_runs", "max_row_nnz") + (("covered_pairs",) if plan_id >= 0 else ()):
            assert ia[key] == ib[key], key
        assert abs(ia["density"] - ib["density"]) < 1e-12 and ib["device_status"] == 0 and ib["layout"] == 1
        with pytest.raises(bsa.BsaError) as e:
            batched.export_csr()
        assert e.value.status == 2
    with pytest.raises(bsa.BsaError) as e:       # heads must be a multiple of the batch size
        bsa.plan_create(mask, *args, layout="nhd", batch=4, **kw)
    assert e.value.status == 1


def test_token_major_layout_from_host_buffers_and_cache_key():
    req = I.config_tiny()
    mask, q, k, v, qkv_cpu = Hh.to_dev(req)
    args = (req.B_Q, req.B_KV, req.N, req.H, req.d)
    with bsa.plan_create(mask, *args) as plan:
        O, LSE = plan.forward(q, k, v)
        torch.cuda.synchronize()
    qh, kh, vh = (t.permute(1, 0, 2).contiguous() for t in qkv_cpu)
    Oh = torch.empty_like(qh)
    Lh = torch.empty((req.H, req.N), dtype=torch.float32)
    bsa.request_host(req.mask, *args, qh, kh, vh, Oh, Lh, layout="nhd")
    assert torch.equal(Oh.permute(1, 0, 2), O.cpu()) and torch.equal(Lh, LSE.cpu())
    cache = bsa.PlanCache(4)
    p0, h0 = cache.get(mask, *args)
    p1, h1 = cache.get(mask, *args, layout="nhd")   # another tensor property: another plan
    p2, h2 = cache.get(mask, *args, layout="nhd")
    assert (h0, h1, h2) == (False, False, True) and p1._h.value == p2._h.value != p0._h.value
    for p in (p0, p1, p2):
        p.destroy()
    cache.destroy()


def test_single_call_request_equals_create_plus_forward():
    req = I.config_tiny()
    mask, q, k, v, qkv_cpu = Hh.to_dev(req)
    args = (req.B_Q, req.B_KV, req.N, req.H, req.d)
    n0 = bsa.kernel_launch_count()
    plan, O, LSE = bsa.request(mask, *args, q, k, v, plan_id=2)
    torch.cuda.synchronize()
    assert bsa.kernel_launch_count() - n0 == 7       # five planner kernels, attention, Split-K merge
    Hh.compare_with_oracle(req, O, LSE, qkv_cpu)
    Hh.check_plan_structure(req, plan)
    with bsa.plan_create(mask, *args, plan_id=2) as two:
        O2, L2 = two.forward(q, k, v)
        O3, L3 = plan.forward(q, k, v)              # the returned plan is an ordinary one
        torch.cuda.synchronize()
    assert torch.equal(O, O2) and torch.equal(LSE, L2) and torch.equal(O, O3) and torch.equal(LSE, L3)
    plan.destroy()
    bits, stride = bsa.pack_mask(mask)
    pb, Ob, Lb = bsa.request(bits, *args, q, k, v, plan_id=2, row_stride=stride)
    torch.cuda.synchronize()
    assert torch.equal(Ob, O) and torch.equal(Lb, LSE)
    pb.destroy()
    with pytest.raises(bsa.BsaError) as e:           # a misaligned tensor is refused before anything is planned
        bsa.request(mask, *args, q.view(-1)[1:1 + q.numel() - 8].view(-1), k, v, O, LSE)
    assert e.value.status == 1


def test_concurrent_requests_from_several_host_threads():
    """Four host threads, each with its own stream, plan and run different requests at the same time (the binding
    releases the interpreter lock inside the C calls; the library keeps its per-request host state per thread), some
    through one shared plan cache: every output equals the one the request gives alone."""
    import threading
    reqs = []
    for t in range(4):
        r = I.config_tiny(seed=40 + t)
        reqs.append((r, Hh.to_dev(r)))
    want = []
    for r, (mask, q, k, v, _) in reqs:
        with bsa.plan_create(mask, r.B_Q, r.B_KV, r.N, r.H, r.d) as plan:
            O, L = plan.forward(q, k, v)
            torch.cuda.synchronize()
            want.append((O.clone(), L.clone()))
    cache = bsa.PlanCache(8)
    errors = []

    def worker(t):
        try:
            r, (mask, q, k, v, _) = reqs[t]
            st = torch.cuda.Stream()
            for it in range(25):
                if it % 2:
                    plan, _ = cache.get(mask, r.B_Q, r.B_KV, r.N, r.H, r.d, stream=st)
                else:
                    plan = bsa.plan_create(mask, r.B_Q, r.B_KV, r.N, r.H, r.d, stream=st)
                O = torch.empty_like(q)
                L = torch.empty(q.shape[:2], dtype=torch.float32, device="cuda")
                plan.forward(q, k, v, O, L, stream=st)
                st.synchronize()
                if not (torch.equal(O, want[t][0]) and torch.equal(L, want[t][1])):
                    errors.append((t, it, "output differs"))
                plan.destroy()
        except Exception as e:  # noqa: BLE001 - reported by the main thread
            errors.append((t, repr(e)))

    torch.cuda.synchronize()
    threads = [threading.Thread(target=worker, args=(t,)) for t in range(4)]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    assert not errors, errors[:3]
    st = cache.stats()
    assert st["hits"] + st["misses"] == 48 and st["entries"] == 4 and st["misses"] >= 4
    cache.destroy()


def test_head_sharded_forward_equals_the_unsharded_one():
    """Heads are independent: three ranks' worth of head ranges, run one after the other on this GPU through the
    sharded driver, give the same bits as the whole request under the same plan."""
    from paper_2609_25869_b200 import shard
    req = I.config_tiny()
    H = 5
    M = I.random_mask(71, H, req.nQb, req.nKb, 0.3, empty_rows=0.1)
    req = I.Request("sharded", H, req.N, req.d, req.B_Q, req.B_KV, M, qkv_seed=29)
    mask, q, k, v, qkv_cpu = Hh.to_dev(req)
    with bsa.plan_create(mask, req.B_Q, req.B_KV, req.N, H, req.d, plan_id=22) as plan:
        O, LSE = plan.forward(q, k, v)
        torch.cuda.synchronize()
    Hh.compare_with_oracle(req, O, LSE, qkv_cpu)
    parts = []
    for lo, hi in shard.head_ranges(H, 3):
        Ol, Ll, info = shard.forward_local(mask[lo:hi].contiguous(), q[lo:hi].contiguous(), k[lo:hi].contiguous(),
                                           v[lo:hi].contiguous(), req.B_Q, req.B_KV, req.N, req.d, plan_id=22)
        assert info["heads"] == hi - lo
        parts.append((Ol, Ll))
    assert torch.equal(torch.cat([p[0] for p in parts]), O) and torch.equal(torch.cat([p[1] for p in parts]), LSE)
    E, L0, none = shard.forward_local(mask[:0], q[:0], k[:0], v[:0], req.B_Q, req.B_KV, req.N, req.d)
    assert E.shape[0] == 0 and L0.shape == (0, req.N) and none is None


# ---------------------------------------------------------------- seeded random requests
def _random_request(n):
    """Request n of a seeded family: geometry, token counts (ragged, N_q != N_kv in a third of the cases), head
    dimension (64, 128 and now and then 256), element type, mask structure (Bernoulli, runs, banded, with empty rows) and plan all follow from n."""
    r = np.random.RandomState(1000 + n)
    B_Q, B_KV = (int(2 ** r.randint(4, 9)) for _ in range(2))
    d = int(r.choice([64, 128]))
    dtype = "fp16" if r.rand() < 0.3 else "bf16"
    H = int(r.randint(1, 5))
    N = int(r.randint(1, 5000))
    N_kv = int(r.randint(1, 5000)) if r.rand() < 0.35 else 0
    nQb, nKb = I.cdiv(N, B_Q), I.cdiv(N_kv or N, B_KV)
    kind = r.randint(0, 3)
    if kind == 0:
        M = I.random_mask(n, H, nQb, nKb, float(r.choice([0.05, 0.3, 0.7, 1.0])), empty_rows=float(r.choice([0.0, 0.2])))
    elif kind == 1:   # a band around the (scaled) diagonal plus a few full columns
        i, j = np.meshgrid(np.arange(nQb), np.arange(nKb), indexing="ij")
        band = np.abs(i * nKb - j * nQb) <= int(r.randint(1, 4)) * max(nQb, nKb)
        M = np.repeat(band[None], H, axis=0).astype(np.uint8)
        M[:, :, r.randint(0, nKb, size=2)] = 1
    else:             # contiguous runs
        M = np.zeros((H, nQb, nKb), dtype=np.uint8)
        for h in range(H):
            for q in range(nQb):
                for _ in range(int(r.randint(0, 4))):
                    a = int(r.randint(0, nKb))
                    M[h, q, a:a + int(r.randint(1, 9))] = 1
    if dtype == "bf16" and r.rand() < 0.12:
        d = 256     # served by the single-tile kernels only
    cat = bsa.catalog()
    ok = [c["plan_id"] for c in cat if bsa.plan_eligible(c["plan_id"], B_Q, B_KV, N, H, d, N_kv=N_kv, dtype=dtype)]
    plan_id = -1 if r.rand() < 0.3 else int(r.choice(ok))
    return I.Request(f"random{n}", H, N, d, B_Q, B_KV, M, qkv_seed=300 + n, N_kv=N_kv, dtype=dtype), plan_id


@pytest.mark.parametrize("n", range(96))
def test_random_requests_match_the_oracle(n):
    req, plan_id = _random_request(n)
    nsel = min(req.nQb, max(1, 600 // req.B_Q))
    Hh.run_request(req, plan_id=plan_id, sel=_sample(req, nsel), guards=False)
    if n % 3:
        return
    # every third request also in the token-major layout, from a bit-packed mask and through the single-call entry
    # point: the same bits as the plain path
    mask, q, k, v, _ = Hh.to_dev(req)
    kw = dict(plan_id=plan_id, N_kv=req.N_kv, dtype=req.dtype)
    args = (req.B_Q, req.B_KV, req.N, req.H, req.d)
    with bsa.plan_create(mask, *args, **kw) as plain:
        O, L = plain.forward(q, k, v)
        torch.cuda.synchronize()
    bits, stride = bsa.pack_mask(mask)
    qt, kt, vt = (t.permute(1, 0, 2).contiguous() for t in (q, k, v))
    pt, Ot, Lt = bsa.request(bits, *args, qt, kt, vt, layout="nhd", row_stride=stride, **kw)
    torch.cuda.synchronize()
    assert pt.info()["device_status"] == 0
    pt.destroy()
    assert torch.equal(Ot.permute(1, 0, 2), O) and torch.equal(Lt, L)


def test_plan_cache_reuses_the_plan_of_a_repeated_mask():
    """Warm path: the second request with the same mask gets the SAME prepared plan (one statistics kernel and one
    row scan launched, nothing else), its output matches the oracle and an uncached plan bit for bit; any change of
    the activity pattern (one block more, one block moved along its row, two rows exchanged) misses."""
    req = I.config_tiny()
    mask, q, k, v, qkv_cpu = Hh.to_dev(req)
    cache = bsa.PlanCache(capacity=8)
    args = (req.B_Q, req.B_KV, req.N, req.H, req.d)
    p0, hit0 = cache.get(mask, *args)
    n0 = bsa.kernel_launch_count()
    p1, hit1 = cache.get(mask.clone(), *args)       # another buffer, the same pattern
    n1 = bsa.kernel_launch_count()
    assert (hit0, hit1) == (False, True) and p0._h.value == p1._h.value
    assert n1 - n0 == 2
    O1, L1 = p1.forward(q, k, v)
    torch.cuda.synchronize()
    Hh.compare_with_oracle(req, O1, L1, qkv_cpu)
    Hh.check_plan_structure(req, p1)
    with bsa.plan_create(mask, *args) as fresh:
        O2, L2 = fresh.forward(q, k, v)
        torch.cuda.synchronize()
        assert torch.equal(O1, O2) and torch.equal(L1, L2)
    # a mask given as other non-zero byte values is the same activity pattern
    p2, hit2 = cache.get(mask * 7, *args)
    assert hit2 and p2._h.value == p0._h.value
    # changed patterns
    M = req.mask.copy()
    h, r = 1, 3
    c_off = int(np.flatnonzero(M[h, r] == 0)[0])
    c_on = int(np.flatnonzero(M[h, r])[0])
    more = M.copy(); more[h, r, c_off] = 1
    moved = more.copy(); moved[h, r, c_on] = 0          # same count as M, one block at another column
    swapped = M.copy(); swapped[h, [r, r + 1]] = swapped[h, [r + 1, r]]
    assert not np.array_equal(swapped, M)
    for variant in (more, moved, swapped):
        pv, hitv = cache.get(torch.from_numpy(variant).cuda(), *args)
        assert not hitv and pv._h.value != p0._h.value
        rv = I.Request("variant", req.H, req.N, req.d, req.B_Q, req.B_KV, variant, qkv_seed=req.qkv_seed)
        Hh.check_plan_structure(rv, pv)
        Ov, Lv = pv.forward(q, k, v)
        torch.cuda.synchronize()
        Hh.compare_with_oracle(rv, Ov, Lv, qkv_cpu)
        pv.destroy()
    # the request key is part of the cache key: another forced plan, or the bit-packed form, is prepared anew
    p3, hit3 = cache.get(mask, *args, plan_id=2)
    bits, stride = bsa.pack_mask(mask)
    p4, hit4 = cache.get(bits, *args, row_stride=stride)
    p5, hit5 = cache.get(bits.clone(), *args, row_stride=stride)
    assert not hit3 and not hit4 and hit5 and p4._h.value == p5._h.value
    O4, L4 = p5.forward(q, k, v)
    torch.cuda.synchronize()
    assert torch.equal(O4, O1) and torch.equal(L4, L1)
    st = cache.stats()
    assert st == {"hits": 3, "misses": 6, "evictions": 0, "entries": 6}
    # get + forward in one call
    O6 = torch.empty_like(q)
    L6 = torch.empty_like(L1)
    n0 = bsa.kernel_launch_count()
    p6, hit6 = cache.request(mask, *args, q, k, v, O6, L6)
    torch.cuda.synchronize()
    assert hit6 and p6._h.value == p0._h.value and bsa.kernel_launch_count() - n0 == 2 + 2   # + attention and merge
    assert torch.equal(O6, O1) and torch.equal(L6, L1)
    for p in (p0, p1, p2, p3, p4, p5, p6):
        p.destroy()
    cache.destroy()


def test_plan_cache_evicts_the_least_recently_used_plan_and_plans_outlive_it():
    req = I.config_tiny()
    _, q, k, v, qkv_cpu = Hh.to_dev(req)
    args = (req.B_Q, req.B_KV, req.N, req.H, req.d)
    masks = []
    for s in range(3):
        masks.append(I.random_mask(100 + s, req.H, req.nQb, req.nKb, 0.25))
    dev = [torch.from_numpy(m).cuda() for m in masks]
    cache = bsa.PlanCache(capacity=2)
    pa, _ = cache.get(dev[0], *args)
    pb, _ = cache.get(dev[1], *args)
    pa2, hit = cache.get(dev[0], *args)            # 0 becomes the most recent
    assert hit
    pc, _ = cache.get(dev[2], *args)               # evicts 1
    assert cache.stats()["evictions"] == 1 and cache.stats()["entries"] == 2
    _, hit_b = cache.get(dev[1], *args)            # prepared again, evicts 0
    _, hit_a = cache.get(dev[0], *args)
    assert not hit_b and not hit_a
    # pb was evicted while held: it is still a complete plan
    rb = I.Request("evicted", req.H, req.N, req.d, req.B_Q, req.B_KV, masks[1], qkv_seed=req.qkv_seed)
    Ob, Lb = pb.forward(q, k, v)
    torch.cuda.synchronize()
    Hh.compare_with_oracle(rb, Ob, Lb, qkv_cpu)
    # plans outlive the cache itself
    cache.destroy()
    ra = I.Request("kept", req.H, req.N, req.d, req.B_Q, req.B_KV, masks[0], qkv_seed=req.qkv_seed)
    Oa, La = pa.forward(q, k, v)
    torch.cuda.synchronize()
    Hh.compare_with_oracle(ra, Oa, La, qkv_cpu)
    for p in (pa, pa2, pb, pc):
        p.destroy()


def test_plan_cache_hit_on_another_stream_waits_for_the_preparation():
    req = I.config_mid()
    mask, q, k, v, _ = Hh.to_dev(req)
    args = (req.B_Q, req.B_KV, req.N, req.H, req.d)
    cache = bsa.PlanCache(capacity=2)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    p0, _ = cache.get(mask, *args, stream=s1)
    p1, hit = cache.get(mask, *args, stream=s2)    # the preparation on s1 may still be running
    assert hit
    with torch.cuda.stream(s2):
        O1 = torch.empty_like(q)
        L1 = torch.empty(q.shape[:2], dtype=torch.float32, device="cuda")
        p1.forward(q, k, v, O1, L1, stream=s2)
    torch.cuda.synchronize()
    with bsa.plan_create(mask, *args) as fresh:
        O2, L2 = fresh.forward(q, k, v)
        torch.cuda.synchronize()
    assert torch.equal(O1, O2) and torch.equal(L1, L2)
    p0.destroy(); p1.destroy()
    cache.destroy()


def test_launch_counter_counts_our_kernels():
    req = I.config_tiny()
    mask, q, k, v, _ = Hh.to_dev(req)
    n0 = bsa.kernel_launch_count()
    with bsa.plan_create(mask, req.B_Q, req.B_KV, req.N, req.H, req.d, plan_id=2) as plan:
        n1 = bsa.kernel_launch_count()
        plan.forward(q, k, v)
        n2 = bsa.kernel_launch_count()
    assert n1 - n0 == 5   # row stats, row scan, CSR fill, tile map, organise
    assert n2 - n1 == 2   # attention + Split-K merge


def test_plan_evicted_while_another_stream_still_runs_its_forward():
    """A plan prepared on stream A, hit from the cache on stream B and forwarded there, then given back by both
    callers and evicted by further requests on stream A: the arenas return to the pool in A's order, and A's next
    requests take memory from that pool at once.  The free has to wait for B's forward (an event recorded behind
    every forward on a foreign stream); B's output is compared with the oracle."""
    req = I.config_stress_b()          # a forward of about a millisecond, long enough to still run during the evictions
    mask, q, k, v, qkv_cpu = Hh.to_dev(req)
    args = (req.B_Q, req.B_KV, req.N, req.H, req.d)
    others = [torch.from_numpy(I.random_mask(200 + s, req.H, req.nQb, req.nKb, 0.2)).cuda() for s in range(4)]
    cache = bsa.PlanCache(capacity=1)
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    pa, hit_a = cache.get(mask, *args, stream=sa)
    pb, hit_b = cache.get(mask, *args, stream=sb)
    assert (hit_a, hit_b) == (False, True)
    O = torch.empty_like(q)
    L = torch.empty((req.H, req.N), dtype=torch.float32, device="cuda")
    scratch_o, scratch_l = torch.empty_like(q), torch.empty_like(L)
    pb.forward(q, k, v, O, L, stream=sb)
    pa.destroy()
    pb.destroy()                       # only the cache holds the plan now
    for m in others:                   # each miss evicts the previous plan and prepares a new one from the pool
        p, hit = cache.get(m, *args, stream=sa)
        assert not hit
        p.forward(q, k, v, scratch_o, scratch_l, stream=sa)
        p.destroy()
    torch.cuda.synchronize()
    assert cache.stats()["evictions"] == 4
    Hh.compare_with_oracle(req, O, L, qkv_cpu, sel=_sample(req, 16))
    cache.destroy()


def test_a_bounded_wait_that_runs_out_ends_in_a_status_not_a_hang():
    """The give-up path of the kernels' bounded waits: with the limit shortened to a few milliseconds of SM clocks
    and the first V tile of every CTA withheld (no copy issued, no arrival: nothing can fault), the waits behind that
    tile run out, the launch returns, the plan reports BSA_ERR_DEVICE_TIMEOUT, and the context stays usable: the next
    forward on a fresh plan matches the oracle."""
    req = I.config_tiny()
    mask, q, k, v, _ = Hh.to_dev(req)
    bsa.debug_set_wait_limit(20_000_000)       # about 10 ms
    bsa.debug_withhold_arrival(True)
    try:
        with bsa.plan_create(mask, req.B_Q, req.B_KV, req.N, req.H, req.d, plan_id=22) as plan:
            plan.forward(q, k, v)
            torch.cuda.synchronize()
            assert plan.info()["device_status"] == 6
    finally:
        bsa.debug_withhold_arrival(False)
        bsa.debug_set_wait_limit(0)
    Hh.run_request(req, plan_id=22)
    Hh.run_request(req, plan_id=-1)
