"""GPU parity: the CUDA path through the C ABI against the CPU oracle on the same seeded inputs.
Popcount accumulators bit-exact; decoded fp32 within 1e-6 relative / 1e-7 absolute."""
import dataclasses

import numpy as np
import pytest

from paper_2609_32922_b200 import workloads as wl
import sc_testlib as T

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2609_32922_b200 import build, binding as b
    build.build()
    return b


@pytest.fixture(scope="module")
def sc(binding):
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    s = binding.ScGemm(0)
    yield s
    assert s.device_status() == 0
    s.close()


CORES = [1, 2, 3, 4, 5]   # POPC, carry-save, simple, tensor-core (one SM per tile), tensor-core (pairs of SMs)


def test_row_stats_and_scales(sc, binding, oracle):
    import torch
    A, _ = wl.make_inputs(wl.small_ragged(M=77, K=101, N=5)[0])
    g = sc.row_stats(torch.from_numpy(A).cuda()).cpu().numpy()
    assert np.array_equal(g, oracle.row_absmax(A))


@pytest.mark.parametrize("mode", ["bipolar", "unipolar"])
@pytest.mark.parametrize("tensor_id", [0, 1])
def test_encode_streams_bit_exact(sc, binding, oracle, mode, tensor_id):
    """Every stream bit of both operands equals the oracle's comparator output (ragged lengths for A)."""
    import torch
    w, L_rows = wl.small_ragged(seed=21, M=70, K=75, N=41, mode=mode, Lmin=0, Lmax=70)
    A, W = wl.make_inputs(w)
    X = A if tensor_id == 0 else W
    Lmax = 70
    params = T.gpu_params(binding, w)
    stream_rows, depth = (w.M, w.K) if tensor_id == 0 else (w.N, w.K)
    dL = torch.from_numpy(L_rows).cuda() if tensor_id == 0 else None
    streams, scales = sc.encode(torch.from_numpy(X).cuda(), tensor_id, dL, Lmax, params)
    bits, neg = sc.unpack(streams, stream_rows, depth, Lmax, T.MODES[mode])
    torch.cuda.synchronize()
    bits = bits.cpu().numpy()
    neg = None if neg is None else neg.cpu().numpy()
    m = T.MODES[mode]
    if tensor_id == 0:
        sig = oracle.scales(A, T.SCALES[w.scale_a], "row")
        ref, _, sign = oracle.encode(A, 0, m, Lmax, w.seed, w.stream_id, sigma_row=sig)
        lens = L_rows
    else:
        sig = oracle.scales(W, T.SCALES[w.scale_w], "col")
        ref, _, sign = oracle.encode(W, 1, m, Lmax, w.seed, w.stream_id, sigma_col=sig)
        ref, sign = ref.transpose(1, 0, 2), sign.T          # stream row = column of W
        lens = np.full(w.N, Lmax, np.int32)
    assert np.array_equal(scales.cpu().numpy(), sig)
    for r in range(stream_rows):
        assert np.array_equal(bits[r, :, :lens[r]], ref[r, :, :lens[r]]), r
        if mode == "unipolar":
            assert np.array_equal(neg[r][:, :lens[r]], ref[r, :, :lens[r]] & sign[r][:, None]), r


@pytest.mark.parametrize("core", CORES)
def test_config1_tiny_full(sc, binding, oracle, core):
    w = wl.TINY
    A, W = wl.make_inputs(w)
    P, C = T.gpu_matmul(sc, binding, w, A, W, None, 64, core=core)
    ref = T.oracle_matmul(oracle, w, A, W, np.full(w.M, 64, np.int32))
    assert np.array_equal(P, ref["P"])
    assert T.close_enough(C, ref["C"])


@pytest.mark.parametrize("core", CORES)
@pytest.mark.parametrize("mode", ["bipolar", "unipolar"])
def test_small_ragged_full(sc, binding, oracle, mode, core):
    """Several tiles, ragged tails in M, N and K, per-row lengths from 0 to 100: every entry compared."""
    w, L_rows = wl.small_ragged(seed=11, mode=mode)
    L_rows[:3] = [0, 1, 100]
    A, W = wl.make_inputs(w)
    P, C = T.gpu_matmul(sc, binding, w, A, W, L_rows, 100, core=core)
    ref = T.oracle_matmul(oracle, w, A, W, L_rows)
    assert np.array_equal(P, ref["P"])
    assert T.close_enough(C, ref["C"])
    assert (C[0] == 0).all() and (P[0] == 0).all()


@pytest.mark.parametrize("mode", ["bipolar", "unipolar"])
def test_int8_grid_first_quantisation(sc, binding, oracle, mode):
    """sc_params.quant = SC_QUANT_INT8_THEN_257: boundaries through the int8 grid (Sec. 4.2), streams and counts equal
    the oracle's with the same rule; prepared weights carry the rule."""
    import torch
    w, L_rows = wl.small_ragged(seed=17, mode=mode)
    A, W = wl.make_inputs(w)
    params = T.gpu_params(binding, w)
    params.quant = binding.SC_QUANT_INT8_THEN_257
    dA, dW, dL = torch.from_numpy(A).cuda(), torch.from_numpy(W).cuda(), torch.from_numpy(L_rows).cuda()
    P, C = sc.matmul(dA, dW, dL, 100, params)
    torch.cuda.synchronize()
    ref = T.oracle_matmul(oracle, w, A, W, L_rows, quant=oracle.QUANT_INT8_THEN_257)
    assert np.array_equal(P.cpu().numpy(), ref["P"]) and T.close_enough(C.cpu().numpy(), ref["C"])
    assert not np.array_equal(ref["P"], T.oracle_matmul(oracle, w, A, W, L_rows)["P"])
    prepared = sc.prepare_weights(dW, 100, params)
    ws = sc.workspace(binding.sc_workspace_bytes_prepared(w.M, w.K, w.N, 100, params))
    P2, C2 = torch.empty_like(P), torch.empty_like(C)
    binding.sc_matmul_prepared(sc.ctx, dA, prepared[0], dL, 100, params, P2, C2, ws)
    torch.cuda.synchronize()
    assert torch.equal(P, P2) and torch.equal(C, C2)
    other = T.gpu_params(binding, w)                                 # the direct rule: the record refuses it
    with pytest.raises(binding.ScError):
        binding.sc_matmul_prepared(sc.ctx, dA, prepared[0], dL, 100, other, P2, C2, ws)
    binding.sc_weights_release(prepared[0])


@pytest.mark.parametrize("mode", ["bipolar", "unipolar"])
@pytest.mark.parametrize("M,N", [(1100, 523), (1024, 512)])
def test_sm_pair_core_odd_tiles_and_ragged_edges(sc, binding, oracle, mode, M, N):
    """The two-SM tensor-core core on shapes that stress its tiling: nine row tiles (the last pair has one tile only), a last
    column tile of 11 columns with N not a multiple of 4 (no bulk reductions), lengths from 0 upwards with whole tiles of
    finished rows; and the exact-fit shape.  Every entry against the oracle."""
    w, L_rows = wl.small_ragged(seed=91, M=M, K=100, N=N, mode=mode, Lmin=0, Lmax=56)
    L_rows[:5] = [56, 0, 1, 55, 56]
    L_rows[M // 2:M // 2 + 300] = 0                    # more than two tiles of rows without a stream
    A, W = wl.make_inputs(w)
    P, C = T.gpu_matmul(sc, binding, w, A, W, L_rows, 56, core=5)
    ref = T.oracle_matmul(oracle, w, A, W, L_rows)
    assert np.array_equal(P, ref["P"])
    assert T.close_enough(C, ref["C"])
    assert sc.device_status() == 0


@pytest.mark.parametrize("N", [1024, 1022])
def test_sm_pair_core_whole_tile_pieces(sc, binding, oracle, N):
    """The two-SM core when its pieces are whole tiles (148 equal tiles on 74 CTA pairs: every run ends on a tile edge), which
    overwrite the zeroed outputs with plain stores instead of reductions: 16-byte stores (N = 1024) and, with N not a multiple
    of 4, single-word stores with a ragged last column tile.  A few rows without a stream shorten the last tile, so that some
    pieces are cut there and both epilogue paths meet in one call.  Every entry against the oracle."""
    M = 37 * 256
    w, L_rows = wl.small_ragged(seed=17, M=M, K=32, N=N, mode="bipolar", Lmin=8, Lmax=8)
    L_rows[:] = 8
    A, W = wl.make_inputs(w)
    for zero_rows in (0, 40):
        L = L_rows.copy()
        if zero_rows:
            L[100:100 + zero_rows] = 0
        P, C = T.gpu_matmul(sc, binding, w, A, W, L, 8, core=5)
        ref = T.oracle_matmul(oracle, w, A, W, L)
        assert np.array_equal(P, ref["P"])
        assert T.close_enough(C, ref["C"])
    assert sc.device_status() == 0


@pytest.mark.parametrize("mode", ["bipolar", "unipolar"])
def test_sm_pair_core_cut_pieces_of_consecutive_rows(sc, binding, oracle, mode):
    """The two-SM core on uniform lengths with few tiles (every piece is a cut tile): warps whose 32 rows are consecutive rows
    of the output add each 32 x 32 chunk with one bulk tensor reduction.  The shape puts rows beyond M and columns beyond N
    inside boxes (clipped), N % 32 != 0 with N % 4 == 0, and a block of rows without a stream splits one warp's run (that warp
    takes the row-by-row path) and leaves lanes without a row in the last tile.  Every entry against the oracle."""
    M, N = 1100, 1020
    w, L_rows = wl.small_ragged(seed=23, M=M, K=100, N=N, mode=mode, Lmin=56, Lmax=56)
    L_rows[:] = 56
    L_rows[300:340] = 0
    A, W = wl.make_inputs(w)
    P, C = T.gpu_matmul(sc, binding, w, A, W, L_rows, 56, core=5)
    ref = T.oracle_matmul(oracle, w, A, W, L_rows)
    assert np.array_equal(P, ref["P"])
    assert T.close_enough(C, ref["C"])
    assert sc.device_status() == 0


def test_groups_and_accumulator_workspace(sc, binding, oracle):
    """Lengths per group of 8 rows (last group short); P not requested (accumulators live in the workspace)."""
    w, _ = wl.small_ragged(seed=5, M=150, K=96, N=130)
    A, W = wl.make_inputs(w)
    rng = np.random.default_rng(3)
    L_groups = rng.integers(1, 60, size=(150 + 7) // 8).astype(np.int32)
    L_rows = oracle.expand_lengths(L_groups, 150, 8)
    P, C = T.gpu_matmul(sc, binding, w, A, W, L_groups, 64, group=8, want_P=False)
    ref = T.oracle_matmul(oracle, w, A, W, L_rows)
    assert P is None and T.close_enough(C, ref["C"])


@pytest.mark.parametrize("shape", [(1, 1, 1), (1, 33, 1), (129, 31, 257), (5, 1000, 3)])
def test_degenerate_shapes(sc, binding, oracle, shape):
    M, K, N = shape
    w, L_rows = wl.small_ragged(seed=31, M=M, K=K, N=N, Lmax=40)
    A, W = wl.make_inputs(w)
    P, C = T.gpu_matmul(sc, binding, w, A, W, L_rows, 40)
    ref = T.oracle_matmul(oracle, w, A, W, L_rows)
    assert np.array_equal(P, ref["P"]) and T.close_enough(C, ref["C"])


def test_maximum_length_and_scale_kinds(sc, binding, oracle):
    """Lmax = SC_L_CAP with per-column weight scales and no activation scale."""
    import dataclasses
    w, _ = wl.small_ragged(seed=41, M=9, K=64, N=12)
    w = dataclasses.replace(w, scale_a="none", scale_w="per_row")
    A, W = wl.make_inputs(w)
    A = np.clip(A * 0.4, -1.5, 1.5).astype(np.float32)          # some values beyond [-1, 1]: clamped
    L_rows = np.array([1024, 1023, 1, 0, 512, 33, 32, 31, 1024], dtype=np.int32)
    P, C = T.gpu_matmul(sc, binding, w, A, W, L_rows, 1024)
    ref = T.oracle_matmul(oracle, w, A, W, L_rows)
    assert np.array_equal(P, ref["P"]) and T.close_enough(C, ref["C"])


def test_assign_lengths_matches_oracle(sc, binding, oracle):
    import torch
    rng = np.random.default_rng(8)
    cases = [(wl.VIT_B_QKV_MIXED, None), (wl.DIT_XL_LINEAR, None)]
    for w, _ in cases:
        avg, Lmin, Lmax, group = w.policy
        A, _ = wl.make_inputs(w)
        g = oracle.row_absmax(A)
        L_ref, avg_ref = oracle.assign_lengths(g, group, avg, Lmin, Lmax)
        dA = torch.from_numpy(A).cuda()
        L, realised = sc.assign_lengths(sc.row_stats(dA), group, avg, Lmin, Lmax, want_realized=True)
        assert np.array_equal(L.cpu().numpy(), L_ref)
        assert realised == avg_ref
    for trial in range(8):
        M = int(rng.integers(1, 3000))
        group = int(rng.choice([1, 1, 3, 8]))
        g = np.abs(rng.standard_normal(M)).astype(np.float32)
        Lmin = int(rng.integers(0, 20))
        Lmax = int(rng.integers(Lmin, 1025))
        avg = float(rng.uniform(Lmin, Lmax + 5))
        L_ref, avg_ref = oracle.assign_lengths(g, group, avg, Lmin, Lmax)
        L, realised = sc.assign_lengths(torch.from_numpy(g).cuda(), group, avg, Lmin, Lmax, want_realized=True)
        assert np.array_equal(L.cpu().numpy(), L_ref), (trial, M, group, Lmin, Lmax, avg)
        assert realised == avg_ref
    # all metrics equal, and the explicit ladder rule
    g = np.full(100, 2.0, np.float32)
    L = sc.assign_lengths(torch.from_numpy(g).cuda(), 1, 37.6, 8, 64)
    assert (L.cpu().numpy() == 37).all()
    g = np.abs(rng.standard_normal(500)).astype(np.float32)
    ladder, tau = [256, 128, 64, 32], [0.75, 0.4, 0.1]
    L = sc.ladder_lengths(torch.from_numpy(g).cuda(), 4, ladder, tau)
    assert np.array_equal(L.cpu().numpy(), oracle.ladder_lengths(g, 4, ladder, tau))


def _sampled_parity(sc, binding, oracle, w, A, W, L_groups, Lmax, group, n_rows, n_cols, core=0):
    L_rows = np.full(w.M, Lmax, np.int32) if L_groups is None else oracle.expand_lengths(L_groups, w.M, group)
    P, C = T.gpu_matmul(sc, binding, w, A, W, L_groups, Lmax, group=group, core=core)
    rows, cols = wl.sample_rows_cols(w, L_rows, n_rows, n_cols)
    ref = T.oracle_matmul(oracle, w, A, W, L_rows, rows, cols)
    assert np.array_equal(P[np.ix_(rows, cols)], ref["P"])
    assert T.close_enough(C[np.ix_(rows, cols)], ref["C"])
    return P, C, L_rows


@pytest.mark.parametrize("core", [1, 2, 4, 5])
def test_config2_vit_b_fc1_sampled(sc, binding, oracle, core):
    w = wl.VIT_B_FC1
    A, W = wl.make_inputs(w)
    P, C, _ = _sampled_parity(sc, binding, oracle, w, A, W, None, 128, 1, 24, 48, core=core)
    # properties that hold at any size: counts within [0, K L]; the estimate tracks the float product
    assert P.min() >= 0 and P.max() <= w.K * 128
    exact = A.astype(np.float64) @ W.astype(np.float64)
    sa = np.abs(A).max(1, keepdims=True).astype(np.float64)
    sw = float(np.abs(W).max())
    z = (C - exact) / (sa * sw * np.sqrt(w.K / 128.0))
    assert abs(z.mean()) < 0.01 and 0.5 < z.std() < 1.05


@pytest.mark.parametrize("core", [0, 4, 5])
def test_config3_mixed_precision_sampled(sc, binding, oracle, core):
    w = wl.VIT_B_QKV_MIXED
    A, W = wl.make_inputs(w)
    L_groups, realised = T.policy_lengths(oracle, w, A)
    assert abs(realised - 64.0) < 1.0
    _sampled_parity(sc, binding, oracle, w, A, W, L_groups, 256, 1, 24, 40, core=core)


@pytest.mark.parametrize("core", [0, 4, 5])
def test_config4_dit_grouped_sampled(sc, binding, oracle, core):
    w = wl.DIT_XL_LINEAR
    A, W = wl.make_inputs(w)
    L_groups, realised = T.policy_lengths(oracle, w, A)
    assert abs(realised - 96.0) < 1.0
    _sampled_parity(sc, binding, oracle, w, A, W, L_groups, 512, 8, 12, 24, core=core)


@pytest.mark.parametrize("L", [8, 32, 128, 512, 1023])
@pytest.mark.parametrize("which", [0, 1, 2, 3])        # qkv, proj, fc1 (bipolar), fc2 (unipolar)
def test_config5_vit_l_sweep_sampled(sc, binding, oracle, which, L):
    """All twenty (layer shape, L) cells of the ViT-L/14 sweep at full size with the default core, each on sampled
    rows x columns evaluated by the oracle."""
    w = wl.vit_l_layers(L)[which]
    A, W = wl.make_inputs(w)
    _sampled_parity(sc, binding, oracle, w, A, W, None, L, 1, 8, 16, core=0)


@pytest.mark.parametrize("which,L", [(1, 32), (3, 128)])
def test_config5_cells_on_the_integer_core(sc, binding, oracle, which, L):
    w = wl.vit_l_layers(L)[which]
    A, W = wl.make_inputs(w)
    _sampled_parity(sc, binding, oracle, w, A, W, None, L, 1, 8, 16, core=2)


def test_row_independence_and_prefix_on_gpu(sc, binding):
    """Row i of a ragged run equals row i of a uniform run at L_i, and shorter streams are prefixes:
    P at length L' is reproduced by a fresh run capped at L' (early termination)."""
    w, L_rows = wl.small_ragged(seed=13, M=300, K=128, N=200, Lmax=90)
    A, W = wl.make_inputs(w)
    P, _ = T.gpu_matmul(sc, binding, w, A, W, L_rows, 90)
    for L in (17, 64):
        Pu, _ = T.gpu_matmul(sc, binding, w, A, W, None, L)
        sel = np.nonzero(L_rows == L)[0]
        assert sel.size > 0
        assert np.array_equal(P[sel], Pu[sel])
    # a row permutation of A permutes the result rows only if streams follow the element index:
    # here streams are keyed by (row, col), so instead check invariance to the tiling order via groups
    P2, _ = T.gpu_matmul(sc, binding, w, A, W, L_rows, 128)        # larger cap, same lengths
    assert np.array_equal(P, P2)


def test_device_detected_errors(sc, binding):
    import torch
    w, L_rows = wl.small_ragged(seed=3, M=40, K=64, N=30, Lmax=20)
    A, W = wl.make_inputs(w)
    bad = A.copy()
    bad[7, 3] = np.nan
    T.gpu_matmul(sc, binding, w, bad, W, L_rows, 20)
    assert sc.device_status() == binding.SC_ERR_NONFINITE
    assert sc.device_status() == 0                                  # cleared by the read
    Lbad = L_rows.copy()
    Lbad[5] = 21
    T.gpu_matmul(sc, binding, w, A, W, Lbad, 20)
    assert sc.device_status() == binding.SC_ERR_LENGTH
    g = torch.ones(10, device="cuda")
    sc.assign_lengths(g, 1, 3.0, 8, 64)
    assert sc.device_status() == binding.SC_ERR_BUDGET
    # host-detected: workspace too small, misaligned, Lmax beyond the cap
    dA, dW = torch.from_numpy(A).cuda(), torch.from_numpy(W).cuda()
    C = torch.empty((40, 30), device="cuda")
    p = T.gpu_params(binding, w)
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.ScError) as e:
        binding.sc_matmul(sc.ctx, dA, dW, None, 20, p, None, C, ws)
    assert e.value.code == binding.SC_ERR_WORKSPACE
    with pytest.raises(binding.ScError) as e:
        binding.sc_matmul(sc.ctx, dA, dW, None, 2000, p, None, C, ws)
    assert e.value.code == binding.SC_ERR_LENGTH


def test_bounded_wait_runs_out_and_the_context_survives(sc, binding, oracle):
    """Failure detection without a fault: a wait of the tensor-core core's own wait routine on a barrier that is never
    signalled gives up after its (here short) clock limit, records SC_ERR_TIMEOUT and the wait site, the second role
    leaves through the abort flag, the kernel returns within milliseconds and the next product is bit-exact."""
    import time
    limit = 1_000_000                                             # SM clocks: about half a millisecond
    binding.sc_selftest_bounded_wait(sc.ctx, 1000)                # first launch loads the kernel's code
    assert sc.device_status() == binding.SC_ERR_TIMEOUT
    t0 = time.perf_counter()
    site, cycles = binding.sc_selftest_bounded_wait(sc.ctx, limit)
    seconds = time.perf_counter() - t0
    assert site[0] & 0xFF == 99 and (site[0] >> 8) & 0xFF == 0 and site[0] >> 16 == 0 and site[1:] == (1, 2)
    assert limit < cycles[0] < 20 * limit                         # gave up after the limit, not much later
    assert 0 < cycles[1] < 30 * limit                             # the other role left through the abort flag
    assert seconds < 0.5
    assert sc.device_status() == binding.SC_ERR_TIMEOUT
    assert sc.device_status() == 0                                # cleared by the read, site slots too
    w, L_rows = wl.small_ragged(seed=11, mode="bipolar")
    A, W = wl.make_inputs(w)
    P, C = T.gpu_matmul(sc, binding, w, A, W, L_rows, 100, core=4)
    ref = T.oracle_matmul(oracle, w, A, W, L_rows)
    assert np.array_equal(P, ref["P"]) and T.close_enough(C, ref["C"])
    assert sc.device_status() == 0


@pytest.mark.parametrize("core", [0, 4])
def test_tensor_core_headroom_fallback(sc, binding, oracle, core):
    """K * Lmax above 2^24 is beyond the exact-integer range of the tensor-core core's fp32 accumulators: the
    automatic choice and an explicit request both fall back to an ALU core, results unchanged."""
    K = 16401
    assert K * 1023 > (1 << 24)
    w, _ = wl.small_ragged(seed=51, M=4, K=K, N=5, Lmax=1023)
    A, W = wl.make_inputs(w)
    L_rows = np.array([1023, 0, 17, 300], dtype=np.int32)
    P, C = T.gpu_matmul(sc, binding, w, A, W, L_rows, 1023, core=core)
    ref = T.oracle_matmul(oracle, w, A, W, L_rows)
    assert np.array_equal(P, ref["P"]) and T.close_enough(C, ref["C"])


@pytest.mark.parametrize("core", [4, 5])
@pytest.mark.parametrize("mode", ["bipolar", "unipolar"])
def test_tensor_core_counts_exact_at_the_headroom_limit(sc, binding, mode, core):
    """K * Lmax = 2^24 exactly, operands at +-1 so that every stream bit is known in closed form (a value of +1 is the
    all-ones stream; -1 is all zeros in bipolar mode and all ones with a negative sign in unipolar mode).  The counts
    reach 2^24 (bipolar) or +-2^23 (unipolar): the largest sums the tensor-core core's fp32 accumulators must hold exactly."""
    K, L, M, N = 16384, 1024, 130, 200
    assert K * L == 1 << 24
    w, _ = wl.small_ragged(seed=71, M=M, K=K, N=N, Lmax=L, mode=mode)
    w = dataclasses.replace(w, scale_a="none", scale_w="none")
    A = np.ones((M, K), dtype=np.float32)
    W = np.ones((K, N), dtype=np.float32)
    W[K // 2:, 1::2] = -1.0               # odd columns: the second half of the depth at -1
    A[1::3, : K // 4] = -1.0              # every third row: the first quarter of the depth at -1
    L_rows = np.full(M, L, dtype=np.int32)
    L_rows[5] = 1000
    P, C = T.gpu_matmul(sc, binding, w, A, W, L_rows, L, core=core)
    # signs: s_a[i][d] * s_w[d][j] summed over d, per position
    sa = np.where(A < 0, -1, 1).astype(np.int64)
    sw = np.where(W < 0, -1, 1).astype(np.int64)
    dot = sa @ sw                                                 # in [-K, K]
    if mode == "bipolar":
        # XNOR of constant streams: 1 where the signs agree
        agree = (K + dot) // 2
        expect = agree * L_rows[:, None].astype(np.int64)
        value = (2 * agree - K).astype(np.float64)
    else:
        expect = dot * L_rows[:, None].astype(np.int64)
        value = dot.astype(np.float64)
    assert np.abs(expect).max() == 1 << 24
    assert np.array_equal(P.astype(np.int64), expect)
    assert np.array_equal(C.astype(np.float64), value)


def test_step_replayed_as_cuda_graph(sc, binding, oracle):
    """The whole step (row statistics, length assignment, SC matmul) is a fixed sequence of asynchronous launches:
    captured once into a CUDA graph and replayed on new inputs it must give what the direct calls give."""
    import torch
    w, _ = wl.small_ragged(seed=61, M=300, K=96, N=200, Lmax=48)
    A, W = wl.make_inputs(w)
    params = T.gpu_params(binding, w, 1, 0)
    dA, dW = torch.from_numpy(A).cuda(), torch.from_numpy(W).cuda()
    g = torch.empty(w.M, dtype=torch.float32, device="cuda")
    L = torch.empty(w.M, dtype=torch.int32, device="cuda")
    P = torch.empty((w.M, w.N), dtype=torch.int32, device="cuda")
    C = torch.empty((w.M, w.N), dtype=torch.float32, device="cuda")
    ws = sc.workspace(binding.sc_workspace_bytes(w.M, w.K, w.N, 48, params))

    def step():
        binding.sc_row_stats(sc.ctx, dA, g)
        binding.sc_assign_lengths(sc.ctx, g, 1, 24.0, 4, 48, L)
        binding.sc_matmul(sc.ctx, dA, dW, L, 48, params, P, C, ws)

    step()                                   # warm-up outside the capture (function attributes, tensor maps)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    rng = np.random.default_rng(5)
    for _ in range(2):
        A2 = (A * rng.uniform(0.2, 3.0, size=(w.M, 1))).astype(np.float32)        # new row ranges -> new lengths
        dA.copy_(torch.from_numpy(A2))
        P.zero_(); C.zero_()
        graph.replay()
        torch.cuda.synchronize()
        L_rows, _ = oracle.assign_lengths(oracle.row_absmax(A2), 1, 24.0, 4, 48)
        assert np.array_equal(L.cpu().numpy(), L_rows)
        ref = T.oracle_matmul(oracle, w, A2, W, L_rows)
        assert np.array_equal(P.cpu().numpy(), ref["P"]) and T.close_enough(C.cpu().numpy(), ref["C"])


@pytest.mark.parametrize("core", [0, 2])
def test_all_rows_without_a_stream(sc, binding, oracle, core):
    """Every length zero: no work unit exists at all; counts and decoded values are zero."""
    w, _ = wl.small_ragged(seed=71, M=130, K=64, N=70, Lmax=16)
    A, W = wl.make_inputs(w)
    L_rows = np.zeros(130, dtype=np.int32)
    P, C = T.gpu_matmul(sc, binding, w, A, W, L_rows, 16, core=core)
    assert (P == 0).all() and (C == 0).all()


def test_selected_tensor_core_kernel_is_reported(sc, binding):
    """`sc_last_core_selected`: forced choices are reported as forced, the integer cores report 0, and under AUTO the plan picks the
    two-SM kernel for long uniform streams and the one-SM kernel for a few positions per row (both decided on the device from
    the lengths), with identical counts either way."""
    w, L_rows = wl.small_ragged(seed=61, M=1024, K=1024, N=1024, mode="bipolar", Lmin=96, Lmax=96)
    A, W = wl.make_inputs(w)
    L_long = np.full(1024, 96, dtype=np.int32)
    L_short = np.full(1024, 2, dtype=np.int32)
    seen = {}
    for core, L in ((4, L_long), (5, L_long), (2, L_long), (0, L_long), (0, L_short)):
        P, _ = T.gpu_matmul(sc, binding, w, A, W, L, 96, core=core)
        seen[(core, int(L[0]))] = (binding.sc_last_core_selected(sc.ctx), P)
    assert seen[(4, 96)][0] == 0 and seen[(5, 96)][0] == 1 and seen[(2, 96)][0] == 0
    assert seen[(0, 96)][0] == 1 and seen[(0, 2)][0] == 0
    for key in ((5, 96), (2, 96), (0, 96)):
        assert np.array_equal(seen[(4, 96)][1], seen[key][1]), key
    assert sc.device_status() == 0


@pytest.mark.parametrize("name", ["vit_b16_fc1", "vit_b16_qkv_mixed", "dit_xl2_linear_grouped", "vit_l14_fc2_L32"])
def test_cores_agree_on_every_output_and_repeat(sc, binding, oracle, name):
    """Full-size runs: the tensor-core core and the carry-save integer core share no code after the encode, so
    every one of their M x N counts must agree (the oracle checks a sample of them elsewhere), and repeating
    the tensor-core call must reproduce its outputs bit for bit (its work items meet through integer reductions)."""
    import torch
    w = wl.all_configs()[name]
    A, W = wl.make_inputs(w)
    if w.policy:
        L_groups, _ = T.policy_lengths(oracle, w, A)
        Lmax, group = w.policy[2], w.policy[3]
    else:
        L_groups, Lmax, group = None, w.uniform_L, 1
    dA, dW = torch.from_numpy(A).cuda(), torch.from_numpy(W).cuda()
    dL = None if L_groups is None else torch.from_numpy(np.ascontiguousarray(L_groups, dtype=np.int32)).cuda()
    outs = []
    for core in (4, 4, 2, 5, 5, 0):
        P, C = sc.matmul(dA, dW, dL, Lmax, T.gpu_params(binding, w, group, core))
        torch.cuda.synchronize()
        outs.append((P.clone(), C.clone()))
    for k in range(1, len(outs)):                       # one-SM tensor core twice, carry-save, SM pairs twice, automatic choice
        assert torch.equal(outs[0][0], outs[k][0]), k
        assert torch.equal(outs[0][1], outs[k][1]), k   # same decode arithmetic on the same counts
