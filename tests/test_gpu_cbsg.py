"""GPU parity of the Sobol-8 / conditional-generation product (sc_matmul_cbsg) against the oracle's cycle-by-cycle
multiplier: XNOR counts bit-exact, decoded values within 1e-6 relative / 1e-7 absolute."""
import numpy as np
import pytest

from paper_2609_32922_b200 import workloads as wl
import sc_testlib as T

pytestmark = pytest.mark.gpu

NONE, PER_ROW, PER_TENSOR = 0, 1, 2


@pytest.fixture(scope="module")
def binding():
    from paper_2609_32922_b200 import build, binding as b
    build.build()
    return b


@pytest.fixture(scope="module")
def sc(binding):
    s = binding.ScGemm(0)
    yield s
    assert s.device_status() == 0
    s.close()


def _run(sc, binding, A, W, L, Lmax, scale_a, scale_w, seed, stream_id=0, group=1, want_P=True, quant=0, core=0):
    import torch
    params = binding.make_params(mode=0, scale_a=scale_a, scale_w=scale_w, group=group, seed=seed, stream_id=stream_id,
                                 quant=quant, core=core)
    dL = None if L is None else torch.from_numpy(np.ascontiguousarray(L, dtype=np.int32)).cuda()
    P, C = sc.matmul_cbsg(torch.from_numpy(A).cuda(), torch.from_numpy(W).cuda(), dL, Lmax, params, want_P)
    torch.cuda.synchronize()
    return (None if P is None else P.cpu().numpy()), C.cpu().numpy()


@pytest.mark.parametrize("core", [4, 5])
@pytest.mark.parametrize("seed,scale_w", [(3, PER_TENSOR), (4, PER_ROW)])
def test_small_ragged_full(sc, binding, oracle, seed, scale_w, core):
    """Several row tiles, a padded column tile, a depth tail; per-row lengths over the whole range 0..256."""
    rng = np.random.default_rng(seed)
    M, K, N = 203, 70, 150
    A = rng.standard_normal((M, K)).astype(np.float32)
    W = (0.02 * rng.standard_normal((K, N))).astype(np.float32)
    L = rng.integers(0, 257, size=M).astype(np.int32)
    L[:4] = [0, 256, 1, 255]
    P, C = _run(sc, binding, A, W, L, 256, PER_ROW, scale_w, seed, stream_id=2, core=core)
    ref = oracle.matmul_cbsg(A, W, L, PER_ROW, scale_w, seed=seed, stream_id=2)
    assert np.array_equal(P, ref["P"])
    assert T.close_enough(C, ref["C"])
    assert (C[0] == 0).all()


def test_int8_grid_first_as_in_the_papers_datapath(sc, binding, oracle):
    """The fused quantisation of Sec. 4.2 in two steps (int8 grid, then one of the 257 boundaries): counts equal the oracle's
    with the same rule and differ from the direct rule's."""
    rng = np.random.default_rng(12)
    M, K, N = 150, 96, 200
    A = rng.standard_normal((M, K)).astype(np.float32)
    W = (0.02 * rng.standard_normal((K, N))).astype(np.float32)
    L = rng.integers(0, 257, size=M).astype(np.int32)
    P, C = _run(sc, binding, A, W, L, 256, PER_ROW, PER_TENSOR, 6, stream_id=1, quant=binding.SC_QUANT_INT8_THEN_257)
    ref = oracle.matmul_cbsg(A, W, L, PER_ROW, PER_TENSOR, seed=6, stream_id=1, quant=oracle.QUANT_INT8_THEN_257)
    assert np.array_equal(P, ref["P"]) and T.close_enough(C, ref["C"])
    direct = oracle.matmul_cbsg(A, W, L, PER_ROW, PER_TENSOR, seed=6, stream_id=1)
    assert not np.array_equal(P, direct["P"])


def test_groups_uniform_and_exact_full_length(sc, binding, oracle):
    rng = np.random.default_rng(9)
    M, K, N = 64, 32, 40
    # operands on the 1/8 grid: at L = 256 every pair product is exact, so C equals the exact matrix product
    A = (rng.integers(-8, 9, size=(M, K)) / 8.0).astype(np.float32)
    W = (rng.integers(-8, 9, size=(K, N)) / 8.0).astype(np.float32)
    P, C = _run(sc, binding, A, W, None, 256, NONE, NONE, 1)
    ref = oracle.matmul_cbsg(A, W, np.full(M, 256, np.int32), NONE, NONE, seed=1)
    assert np.array_equal(P, ref["P"]) and T.close_enough(C, ref["C"])
    assert np.allclose(C, A.astype(np.float64) @ W.astype(np.float64), rtol=0, atol=1e-5)
    # lengths per group of 8 rows, counts not requested
    Lg = rng.integers(0, 200, size=M // 8).astype(np.int32)
    P2, C2 = _run(sc, binding, A, W, Lg, 199, NONE, NONE, 1, group=8, want_P=False)
    ref2 = oracle.matmul_cbsg(A, W, np.repeat(Lg, 8), NONE, NONE, seed=1)
    assert P2 is None and T.close_enough(C2, ref2["C"])


@pytest.mark.parametrize("core", [0, 5])
def test_vit_b_fc1_sampled(sc, binding, oracle, core):
    """Config-2 shape (1576 x 768 x 3072) at L = 128: sampled rows x columns against the oracle."""
    w = wl.VIT_B_FC1
    A, W = wl.make_inputs(w)
    L = np.full(w.M, 128, dtype=np.int32)
    P, C = _run(sc, binding, A, W, L, 128, PER_ROW, PER_TENSOR, w.seed, core=core)
    rows, cols = wl.sample_rows_cols(w, L, 10, 24)
    ref = oracle.matmul_cbsg(A, W, L, PER_ROW, PER_TENSOR, seed=w.seed, row_sel=rows, col_sel=cols)
    assert np.array_equal(P[np.ix_(rows, cols)], ref["P"])
    assert T.close_enough(C[np.ix_(rows, cols)], ref["C"])


def test_argument_checks(sc, binding):
    import torch
    A = torch.zeros((8, 16), device="cuda"); W = torch.zeros((16, 8), device="cuda")
    C = torch.empty((8, 8), device="cuda")
    p = binding.make_params(mode=0)
    ws = sc.workspace(binding.sc_workspace_bytes_cbsg(8, 16, 8, 256, p))

    def code(Lmax=64, **kw):
        q = binding.make_params(mode=0)
        for k, v in kw.items():
            setattr(q, k, v)
        try:
            binding.sc_matmul_cbsg(sc.ctx, A, W, None, Lmax, q, None, C, ws)
        except binding.ScError as e:
            return e.code
        return 0

    assert code() == 0
    assert code(Lmax=257) == binding.SC_ERR_LENGTH
    assert code(mode=1) == binding.SC_ERR_ARG
    assert code(core=1) == binding.SC_ERR_ARG
    assert binding.sc_workspace_bytes_cbsg(8, 40000, 8, 256, p) == 0     # 2 K Lmax beyond the accumulator headroom
    # out-of-range lengths are found on the device
    L = torch.tensor([5, 300, 7, 1, 1, 1, 1, 1], dtype=torch.int32, device="cuda")
    binding.sc_matmul_cbsg(sc.ctx, A, W, L, 64, p, None, C, ws)
    assert sc.device_status() == binding.SC_ERR_LENGTH


def test_scc_diagnostic_matches_oracle(sc, binding, oracle):
    import torch
    rng = np.random.default_rng(5)
    n = 3000
    Ta = rng.integers(0, 257, size=n).astype(np.int32)
    Tw = rng.integers(0, 257, size=n).astype(np.int32)
    Ta[:4], Tw[:4] = [0, 256, 128, 64], [77, 77, 128, 192]
    ws = sc.workspace(32768)
    for L, seed in ((256, 3), (100, 4), (1, 5), (0, 6)):
        counts = torch.empty((n, 4), dtype=torch.int32, device="cuda")
        scc = torch.empty(n, dtype=torch.float64, device="cuda")
        binding.sc_cbsg_scc(sc.ctx, torch.from_numpy(Ta).cuda(), torch.from_numpy(Tw).cuda(), L, seed, 2, counts, scc, ws)
        torch.cuda.synchronize()
        got_c, got_s = counts.cpu().numpy(), scc.cpu().numpy()
        scr = oracle.cbsg_scramble(seed, 2)
        for i in list(range(8)) + list(rng.integers(0, n, 60)):
            _, ref = oracle.cbsg_pair(int(Ta[i]), int(Tw[i]), L, scr)
            assert got_c[i].tolist() == ref.tolist(), (L, i)
            assert got_s[i] == oracle.scc(*[int(v) for v in ref])
    # on the 1/16 grid at full length the correlation vanishes exactly (Appendix A.1)
    grid = (np.arange(17) * 16).astype(np.int32)
    Ta2, Tw2 = np.repeat(grid, 17), np.tile(grid, 17)
    scc = torch.empty(289, dtype=torch.float64, device="cuda")
    binding.sc_cbsg_scc(sc.ctx, torch.from_numpy(Ta2).cuda(), torch.from_numpy(Tw2).cuda(), 256, 9, 0, None, scc, ws)
    assert (scc.cpu().numpy() == 0).all()
