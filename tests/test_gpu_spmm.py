"""Parity of the CUDA SpMM with the CPU oracle (needs a B200).  Everything goes through the C ABI.

Y is compared element by element with the dense float64 product of the masked W (the plain
definition), within the tolerance of the benchmark spec, |y - y_ref| <= 2e-3 * sum_k |w_ik x_kj|
+ 1e-3, and with the oracle's own format-walking SpMM.  Cases where all partial sums are exactly
representable (identity X, small integers) must match bit for bit.
"""
import numpy as np
import pytest

from paper_2607_08786_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tl3():
    import torch
    assert torch.cuda.is_available()
    from paper_2607_08786_b200 import build, tl3 as mod
    build.build_library()
    mod.lib()                                   # raises if the CUDA library is missing: no fallback
    return mod


def device_X(X, ld=None):
    import torch
    K, N = X.shape
    ld = ld or (N + 7) // 8 * 8
    buf = torch.zeros((K, ld), dtype=torch.float16, device="cuda")
    buf[:, :N] = torch.from_numpy(X)
    return buf[:, :N]


def run_gpu(tl3, W, X, ldx=None, ldy=None, repeats=1):
    import torch
    m = tl3.encode(W)
    m.upload()
    Xd = device_X(X, ldx)
    N = X.shape[1]
    ws = m.new_workspace(N)
    Ybuf = torch.full((W.shape[0], ldy or N), float("nan"), dtype=torch.float16, device="cuda")
    Y = Ybuf[:, :N]
    outs = []
    for _ in range(repeats):
        m.spmm(Xd, Y, workspace=ws)
        torch.cuda.synchronize()
        assert m.status(ws) == tl3.OK
        outs.append(Y.cpu().numpy().copy())
    if ldy and ldy > N:                          # columns beyond N are left alone
        assert torch.isnan(Ybuf[:, N:]).all()
    for o in outs[1:]:
        assert np.array_equal(o.view(np.uint16), outs[0].view(np.uint16))   # deterministic
    return outs[0], m


def check(oracle_mod, W, X, Y, with_oracle_spmm=True):
    Yref, bound = oracle_mod.dense_fp64(W, X)
    err = np.abs(Y.astype(np.float64) - Yref)
    tol = oracle_mod.tolerance(bound)
    assert np.all(err <= tol), f"max err/tol {np.max(err / tol):.3f} at {np.unravel_index(np.argmax(err / tol), err.shape)}"
    if with_oracle_spmm:
        Yo = oracle_mod.spmm(oracle_mod.encode(W), X).view(np.float16).astype(np.float64)
        # both accumulate in fp32 (different order) and round once to fp16
        assert np.all(np.abs(Y.astype(np.float64) - Yo) <= 2.0**-9 * np.abs(Yo) + 1e-4 * bound + 1e-6)


def test_config1(tl3, oracle_mod):
    case = next(wl.config_cases(1))
    W, X = case.make_W(), case.make_X()
    Y, m = run_gpu(tl3, W, X, repeats=3)
    check(oracle_mod, W, X, Y)
    assert m.last_launch()["ctas"] == 64


@pytest.mark.parametrize("N", [1, 5, 8, 16, 24, 32, 48, 64])
def test_all_widths(tl3, oracle_mod, N):
    case = wl.Case(0, "n", 640, 896, N, 40 + N, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    Y, _ = run_gpu(tl3, W, X, repeats=2)
    check(oracle_mod, W, X, Y)


@pytest.mark.parametrize("shape", [(1, 8), (127, 129), (130, 260), (1000, 1096), (384, 128), (128, 4096), (4096, 128)])
def test_ragged_shapes(tl3, oracle_mod, shape):
    case = wl.Case(0, "r", shape[0], shape[1], 16, shape[0] + shape[1], 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    Y, _ = run_gpu(tl3, W, X)
    check(oracle_mod, W, X, Y)


@pytest.mark.parametrize("sparsity,kind", [(0.4, "magnitude"), (0.6, "magnitude"), (0.7, "magnitude"),
                                           (0.5, "wanda"), (0.5, "row_scaled"), (0.5, "bernoulli")])
def test_sparsities_and_masks(tl3, oracle_mod, sparsity, kind):
    case = wl.Case(0, "s", 1536, 2048, 16, int(sparsity * 100), sparsity, kind)
    W, X = case.make_W(), case.make_X()
    Y, _ = run_gpu(tl3, W, X)
    check(oracle_mod, W, X, Y)


def test_split_k_many_and_few_contributors(tl3, oracle_mod):
    # 2 row-tiles x 160 k-tiles: every row-tile is shared by ~74 CTAs
    case = wl.Case(0, "wide", 256, 20480, 8, 77, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    Y, m = run_gpu(tl3, W, X, repeats=2)
    check(oracle_mod, W, X, Y)
    assert m.last_launch()["ctas"] == 148
    # 160 row-tiles x 2 k-tiles: most row-tiles belong to one CTA, some straddle two
    case = wl.Case(0, "tall", 20480, 256, 8, 78, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    Y, _ = run_gpu(tl3, W, X, repeats=2)
    check(oracle_mod, W, X, Y)


def test_degenerate_matrices(tl3, oracle_mod):
    rng = np.random.default_rng(3)
    X = rng.standard_normal((512, 16)).astype(np.float16)
    Z = np.zeros((256, 512), dtype=np.float16)
    Y, _ = run_gpu(tl3, Z, X)
    assert not Y.view(np.uint16).any()                             # all-zero W: exact zeros
    D = (rng.standard_normal((256, 512)) * 0.05).astype(np.float16)   # fully dense: half of nnz is Residual
    D[D == 0] = np.float16(0.01)
    Y, m = run_gpu(tl3, D, X)
    assert m.stats()["n_res"] == D.size // 2
    check(oracle_mod, D, X, Y)
    keep = np.zeros((256, 128, 4), dtype=bool)                        # exact 2:4: only the Sparse-TC layer
    keep[:, :, [0, 3]] = True
    W24 = np.where(keep.reshape(256, 512), D, np.float16(0))
    Y, m = run_gpu(tl3, W24, X)
    assert m.stats()["n_sf"] == 0 and m.stats()["n_res"] == 0
    check(oracle_mod, W24, X, Y)
    T = np.zeros((256, 512), dtype=np.float16)                        # every surplus parked in another row
    T[:64] = D[:64]
    T[128:192] = D[128:192]
    Y, _ = run_gpu(tl3, T, X)
    check(oracle_mod, T, X, Y)


@pytest.mark.parametrize("seed", range(6))
def test_adversarial_density_patterns(tl3, oracle_mod, seed):
    """Density that changes abruptly by row band and column band: tiles with no parked elements,
    tiles that are all Residual, tiles with one, two or three code words per chain, side by side."""
    rng = np.random.default_rng([78, seed])
    M, K, N = 640, 1152, (8, 16, 24, 32, 48, 64)[seed]
    dens_r = rng.choice([0.0, 0.1, 0.5, 0.9, 1.0], size=M // 32).repeat(32)
    dens_c = rng.choice([0.0, 0.25, 0.5, 0.75, 1.0], size=K // 64).repeat(64)
    p = np.clip(0.5 * (dens_r[:, None] + dens_c[None, :]) + rng.choice([-0.3, 0.0, 0.3]), 0, 1)
    W = np.where(rng.random((M, K)) < p, (rng.standard_normal((M, K)) * 0.05).astype(np.float16), np.float16(0))
    W[(W.view(np.uint16) & 0x7FFF) == 0] = 0
    X = rng.standard_normal((K, N)).astype(np.float16)
    Y, _ = run_gpu(tl3, W, X, repeats=2)
    check(oracle_mod, W, X, Y)


def test_device_chain_overflow(tl3, oracle_mod):
    """A tile whose device-image chains overflow into the Residual list (see special_cases)."""
    from special_cases import clustered_surplus_tile
    W = np.tile(clustered_surplus_tile(), (2, 3))
    X = np.random.default_rng(5).standard_normal((384, 16)).astype(np.float16)
    Y, _ = run_gpu(tl3, W, X)
    check(oracle_mod, W, X, Y)


def test_fewer_stages_than_decode_groups(tl3, oracle_mod):
    """Large blocks (heavy Residual layer) and a wide X leave room for only two or three stages in
    shared memory; several tiles per CTA, so the ring wraps many times."""
    case = wl.Case(0, "s3", 4096, 2048, 64, 3, 0.4, "magnitude")
    W, X = case.make_W(), case.make_X()
    Y, m = run_gpu(tl3, W, X, repeats=2)
    assert m.last_launch()["stages"] <= 3
    check(oracle_mod, W, X, Y)
    rng = np.random.default_rng(8)
    D = (rng.standard_normal((2048, 2048)) * 0.05).astype(np.float16)      # fully dense: half of nnz is Residual
    D[D == 0] = np.float16(0.01)
    X = rng.standard_normal((2048, 32)).astype(np.float16)
    Y, m = run_gpu(tl3, D, X, repeats=2)
    assert m.last_launch()["stages"] == 2
    check(oracle_mod, D, X, Y)


def test_workspace_is_left_cleared_and_can_serve_another_matrix(tl3, oracle_mod):
    """The split-K hand-over keeps one flag per partial-sum slot in the workspace and relies on
    finding them all at zero: after a launch the head of the workspace (status word and flags)
    must read zero again, and the same workspace must then serve a different matrix."""
    import torch
    a = wl.Case(0, "ws_a", 1024, 5120, 16, 501, 0.5, "magnitude")      # every row-tile shared by many CTAs
    b = wl.Case(0, "ws_b", 2304, 1152, 16, 502, 0.5, "bernoulli")      # other tile counts, other sharing pattern
    Wa, Xa, Wb, Xb = a.make_W(), a.make_X(), b.make_W(), b.make_X()
    ma, mb = tl3.encode(Wa), tl3.encode(Wb)
    ma.upload()
    mb.upload()
    n = max(ma.workspace_bytes(16), mb.workspace_bytes(16))
    ws = torch.empty(n, dtype=torch.uint8, device="cuda")
    assert tl3.lib().tl3_workspace_init(ws.data_ptr(), n, None) == tl3.OK
    for m, W, X in ((ma, Wa, Xa), (mb, Wb, Xb), (ma, Wa, Xa)):
        Y = m.spmm(device_X(X), workspace=ws)
        torch.cuda.synchronize()
        assert m.status(ws) == tl3.OK
        assert int(ws[:4096].to(torch.int32).sum().item()) == 0
        check(oracle_mod, W, X, Y.cpu().numpy(), with_oracle_spmm=False)


def test_thousands_of_back_to_back_launches(tl3, oracle_mod):
    """Five different launches in one CUDA graph, replayed without host synchronisation: every
    replay must leave the status words clear and reproduce the first result bit for bit (the
    pipeline's barrier protocol must not depend on how loads happen to be ordered in time)."""
    import torch
    cases = [wl.Case(0, "a", 2560, 5120, 16, 1, 0.5, "magnitude"), wl.Case(0, "b", 2048, 8192, 32, 2, 0.5, "magnitude"),
             wl.Case(0, "c", 2048, 2048, 64, 3, 0.4, "magnitude"), wl.Case(0, "d", 1024, 1024, 8, 4, 0.5, "bernoulli"),
             wl.Case(0, "e", 3000, 3000, 24, 5, 0.7, "magnitude")]
    L = []
    for c in cases:
        W, X = c.make_W(), c.make_X()
        m = tl3.encode(W)
        m.upload()
        Xd = device_X(X)
        ws = m.new_workspace(c.N)
        Y = torch.empty((c.M, c.N), dtype=torch.float16, device="cuda")
        m.spmm(Xd, Y, workspace=ws)
        torch.cuda.synchronize()
        check(oracle_mod, W, X, Y.cpu().numpy())             # the result every replay is compared with
        L.append((c, m, Xd, Y, ws, Y.clone()))

    def step():
        for c, m, Xd, Y, ws, ref in L:
            m.spmm(Xd, Y, workspace=ws)

    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    for _ in range(5):
        for _ in range(100):
            g.replay()
        torch.cuda.synchronize()
        for c, m, Xd, Y, ws, ref in L:
            assert m.status_word(ws) == 0, c.name
            assert torch.equal(Y, ref), c.name


def test_concurrent_launches_on_several_streams(tl3, oracle_mod):
    """The same five launches forked over three streams inside one CUDA graph, so that kernels of
    different streams share the GPU (a kernel moves in as another moves out, and CTAs of a launch
    may still be waiting for an SM while its reducers already collect): results and status as in
    the serial run, replay after replay."""
    import torch
    cases = [wl.Case(0, "a", 2560, 5120, 16, 1, 0.5, "magnitude"), wl.Case(0, "b", 2048, 8192, 32, 2, 0.5, "magnitude"),
             wl.Case(0, "c", 2048, 2048, 64, 3, 0.4, "magnitude"), wl.Case(0, "d", 1024, 1024, 8, 4, 0.5, "bernoulli"),
             wl.Case(0, "e", 3000, 3000, 24, 5, 0.7, "magnitude")]
    L = []
    for c in cases:
        W, X = c.make_W(), c.make_X()
        m = tl3.encode(W)
        m.upload()
        Xd = device_X(X)
        ws = m.new_workspace(c.N)
        Y = torch.empty((c.M, c.N), dtype=torch.float16, device="cuda")
        m.spmm(Xd, Y, workspace=ws)
        torch.cuda.synchronize()
        check(oracle_mod, W, X, Y.cpu().numpy())             # the result every replay is compared with
        L.append((c, m, Xd, Y, ws, Y.clone()))
    side = [torch.cuda.Stream() for _ in range(2)]

    def step():
        cur = torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(cur)
        for s in side:
            s.wait_event(start)
        for i, (c, m, Xd, Y, ws, ref) in enumerate(L):
            m.spmm(Xd, Y, workspace=ws, stream=cur if i % 3 == 0 else side[i % 3 - 1])
        for s in side:
            done = torch.cuda.Event()
            done.record(s)
            cur.wait_event(done)

    step()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    for _ in range(5):
        for _ in range(100):
            g.replay()
        torch.cuda.synchronize()
        for c, m, Xd, Y, ws, ref in L:
            assert m.status_word(ws) == 0, c.name
            assert torch.equal(Y, ref), c.name


def test_identity_X_reproduces_W_bit_for_bit(tl3):
    """Each y_ij is one product w_ij * 1: the GPU must hand back the decoded W exactly."""
    for k0 in (0, 64):
        case = wl.Case(0, "id", 512, 128, 64, 90 + k0, 0.5, "magnitude")
        W = case.make_W()
        X = np.zeros((128, 64), dtype=np.float16)
        X[k0:k0 + 64] = np.eye(64, dtype=np.float16)
        Y, _ = run_gpu(tl3, W, X)
        assert np.array_equal(Y.view(np.uint16), W[:, k0:k0 + 64].view(np.uint16))


def test_small_integers_are_exact(tl3, oracle_mod):
    rng = np.random.default_rng(12)
    W = np.where(rng.random((384, 1280)) < 0.5, rng.integers(-4, 5, (384, 1280)), 0).astype(np.float16)
    X = rng.integers(-3, 4, (1280, 32)).astype(np.float16)
    Y, _ = run_gpu(tl3, W, X)
    assert np.array_equal(Y.astype(np.int64), W.astype(np.int64) @ X.astype(np.int64))
    assert np.array_equal(Y.view(np.uint16), oracle_mod.spmm(oracle_mod.encode(W), X))


@pytest.mark.parametrize("N", [72, 128, 200])
def test_wide_activation_blocks(tl3, oracle_mod, N):
    """N > 64 (towards prefill) runs as 64-column blocks."""
    case = wl.Case(0, "wide_n", 512, 768, N, 60 + N, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    Y, _ = run_gpu(tl3, W, X, repeats=2)
    check(oracle_mod, W, X, Y)


@pytest.mark.parametrize("activation", [None, "relu", "silu", "gelu_tanh"])
@pytest.mark.parametrize("shape", [(384, 512, 16), (1000, 1096, 24), (5120, 640, 32)])
def test_bias_and_activation_epilogue(tl3, oracle_mod, activation, shape):
    """Y = act(W X + b) against the same expression in float64 (complete row-tiles, the direct
    write of the last contributor and the reduction of partial sums all pass through it)."""
    import torch
    M, K, N = shape
    case = wl.Case(0, "ep", M, K, N, 31, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    bias = (np.random.default_rng(7).standard_normal(M) * 0.5).astype(np.float16)
    m = tl3.encode(W)
    m.upload()
    Y = m.spmm(device_X(X), bias=torch.from_numpy(bias).cuda(), activation=activation)
    torch.cuda.synchronize()
    Yref, bound = oracle_mod.dense_fp64(W, X)
    z = Yref + bias.astype(np.float64)[:, None]
    if activation == "relu":
        ref = np.maximum(z, 0)
    elif activation == "silu":
        ref = z / (1 + np.exp(-z))
    elif activation == "gelu_tanh":
        ref = 0.5 * z * (1 + np.tanh(np.sqrt(2 / np.pi) * (z + 0.044715 * z ** 3)))
    else:
        ref = z
    # the activations used here have slopes within [-0.13, 1.13]; the output rounding is within the 1e-3 + 2e-3 * bound
    tol = 1.2 * oracle_mod.tolerance(bound + np.abs(bias.astype(np.float64))[:, None]) + 1e-3
    assert (np.abs(Y.cpu().numpy().astype(np.float64) - ref) <= tol).all()
    if activation is None:                          # without a bias and an activation: the plain product, bit for bit
        Y0 = m.spmm(device_X(X))
        Y1 = m.spmm(device_X(X), bias=torch.zeros(M, dtype=torch.float16, device="cuda"))
        torch.cuda.synchronize()
        assert torch.equal(Y0, Y1)


@pytest.mark.parametrize("shape", [(384, 512, 16), (1000, 1096, 5), (130, 260, 24), (5120, 640, 32), (256, 4096, 64), (640, 896, 100)])
def test_transposed_activations(tl3, oracle_mod, shape):
    """Yt = Xt W^T with X and Y in the [batch, hidden] layout: the same numbers as Y = W X, and bit
    for bit the same as the untransposed entry point (same products, same order)."""
    import torch
    M, K, N = shape
    case = wl.Case(0, "nt", M, K, N, 41, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    m = tl3.encode(W)
    m.upload()
    ldk = (K + 7) // 8 * 8
    Xt = torch.zeros((N, ldk), dtype=torch.float16, device="cuda")[:, :K]
    Xt.copy_(torch.from_numpy(np.ascontiguousarray(X.T)))
    Ytbuf = torch.full((N, M + 3), float("nan"), dtype=torch.float16, device="cuda")
    Yt = m.spmm_nt(Xt, Ytbuf[:, :M])
    torch.cuda.synchronize()
    assert torch.isnan(Ytbuf[:, M:]).all()
    Y = Yt.cpu().numpy().T
    check(oracle_mod, W, X, np.ascontiguousarray(Y))
    Y0 = m.spmm(device_X(X))
    torch.cuda.synchronize()
    assert np.array_equal(Y0.cpu().numpy().view(np.uint16), np.ascontiguousarray(Y).view(np.uint16))
    bias = (np.random.default_rng(9).standard_normal(M) * 0.5).astype(np.float16)
    b = torch.from_numpy(bias).cuda()
    Y1 = m.spmm_nt(Xt, bias=b, activation="silu")
    Y2 = m.spmm(device_X(X), bias=b, activation="silu")
    torch.cuda.synchronize()
    assert torch.equal(Y1.T.contiguous(), Y2)


def test_strided_operands(tl3, oracle_mod):
    case = wl.Case(0, "ld", 300, 700, 12, 5, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    Y, _ = run_gpu(tl3, W, X, ldx=40, ldy=19)
    check(oracle_mod, W, X, Y)


def test_argument_errors_on_device(tl3):
    import torch
    case = wl.Case(0, "e", 256, 256, 8, 5, 0.5, "magnitude")
    m = tl3.encode(case.make_W())
    X = torch.zeros((256, 8), dtype=torch.float16, device="cuda")
    Y = torch.zeros((256, 8), dtype=torch.float16, device="cuda")
    L = tl3.lib()
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    assert L.tl3_spmm(m._h, X.data_ptr(), 8, Y.data_ptr(), 8, 8, ws.data_ptr(), None) == tl3.ERR_NOT_UPLOADED
    m.upload()
    ws = m.new_workspace(8)
    assert L.tl3_spmm(m._h, X.data_ptr(), 8, Y.data_ptr(), 8, 4097, ws.data_ptr(), None) == tl3.ERR_UNSUPPORTED
    assert L.tl3_spmm(m._h, X.data_ptr(), 8, Y.data_ptr(), 8, 65, ws.data_ptr(), None) == tl3.ERR_INVALID_ARG   # ldx < N
    assert L.tl3_spmm(m._h, X.data_ptr(), 8, Y.data_ptr(), 8, 0, ws.data_ptr(), None) == tl3.ERR_UNSUPPORTED
    assert L.tl3_spmm(m._h, X.data_ptr(), 12, Y.data_ptr(), 8, 8, ws.data_ptr(), None) == tl3.ERR_INVALID_ARG   # ldx % 8
    assert L.tl3_spmm(m._h, X.data_ptr() + 2, 8, Y.data_ptr(), 8, 8, ws.data_ptr(), None) == tl3.ERR_INVALID_ARG  # X alignment
    assert L.tl3_spmm(m._h, X.data_ptr(), 8, Y.data_ptr(), 4, 8, ws.data_ptr(), None) == tl3.ERR_INVALID_ARG    # ldy < N
    assert L.tl3_spmm(m._h, X.data_ptr(), 8, Y.data_ptr(), 8, 8, ws.data_ptr(), None) == tl3.OK
    torch.cuda.synchronize()
    assert m.status(ws) == tl3.OK


def test_random_shapes_widths_and_masks(tl3, oracle_mod):
    """Forty seeded random problems: ragged M and K, every width from 1 to 80, sparsities 30-90 %,
    all four mask kinds, wide-and-flat and tall-and-thin matrices (many or no CTAs per row-tile).
    Each one twice: within tolerance of the float64 definition, same bits both times, status clear."""
    import torch
    rng = np.random.default_rng(20260)
    for _ in range(40):
        M = int(rng.integers(1, 24)) * 128 + int(rng.choice([0, 0, 0, 1, 37, 64, 127]))
        K = int(rng.integers(1, 24)) * 128 + int(rng.choice([0, 0, 0, 8, 40, 120]))
        if rng.random() < 0.25:
            a, b = int(rng.integers(1, 4)) * 128, int(rng.integers(40, 120)) * 128
            M, K = (a, b) if rng.random() < 0.5 else (b, a)
        N = int(rng.choice([1, 3, 8, 12, 16, 24, 32, 48, 64, 80]))
        case = wl.Case(0, "rnd", M, K, N, int(rng.integers(0, 1 << 30)), float(rng.choice([0.3, 0.4, 0.5, 0.5, 0.6, 0.7, 0.9])),
                       str(rng.choice(["magnitude", "bernoulli", "row_scaled", "wanda"])))
        W, X = case.make_W(), case.make_X()
        Y, m = run_gpu(tl3, W, X, repeats=2)
        check(oracle_mod, W, X, Y, with_oracle_spmm=False)
        m.close()
        torch.cuda.empty_cache()


def test_a_wait_that_nothing_ends_gives_up_and_reports(tl3, oracle_mod):
    """Every wait inside the kernels is bounded.  The library's self-test waits on a barrier that
    nothing arrives at: the kernel must return by itself, the status must say which wait gave up,
    and the device must work as before."""
    import time
    import torch
    case = wl.Case(0, "after_timeout", 512, 1024, 8, 31, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    m = tl3.encode(W)
    m.upload()
    ws = m.new_workspace(case.N)
    stream = torch.cuda.current_stream().cuda_stream
    t0 = time.time()
    assert tl3.lib().tl3_selftest_bounded_wait(ws.data_ptr(), stream) == tl3.OK
    assert m.status(ws) == tl3.ERR_DEVICE_TIMEOUT          # synchronises: returns when the kernel has given up
    assert 1.0 < time.time() - t0 < 30.0
    assert m.status_word(ws) & 0xFF == 1
    assert int(ws[4:8].view(torch.int32).item()) == 2      # the wait gave up, it did not complete
    assert tl3.lib().tl3_workspace_init(ws.data_ptr(), ws.numel(), stream) == tl3.OK
    Y = m.spmm(device_X(X), workspace=ws)
    torch.cuda.synchronize()
    assert m.status(ws) == tl3.OK
    check(oracle_mod, W, X, Y.cpu().numpy(), with_oracle_spmm=False)


def test_host_buffer_entry_point(tl3, oracle_mod):
    import torch
    case = wl.Case(0, "h", 640, 512, 12, 8, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    m = tl3.encode(W)
    m.upload()
    ws = m.new_workspace(case.N)
    dX = torch.empty(case.K * 16 * 2, dtype=torch.uint8, device="cuda")
    dY = torch.empty(case.M * case.N * 2, dtype=torch.uint8, device="cuda")
    Y = np.zeros((case.M, case.N), dtype=np.float16)
    m.spmm_host(X, Y, dX, dY, ws)
    check(oracle_mod, W, X, Y)


def test_host_buffer_entry_point_async_on_several_streams(tl3, oracle_mod):
    """Three products enqueued on three streams (own staging buffers and workspaces), one wait at
    the end: each result equals what the blocking call gives."""
    import torch
    cases = [wl.Case(0, "ha", 1024, 2560, 16, 21, 0.5, "magnitude"), wl.Case(0, "hb", 2560, 1024, 8, 22, 0.5, "magnitude"),
             wl.Case(0, "hc", 640, 512, 12, 23, 0.5, "bernoulli")]
    streams = [torch.cuda.Stream() for _ in cases]
    jobs = []
    for c in cases:
        W, X = c.make_W(), c.make_X()
        m = tl3.encode(W)
        m.upload()
        Xp = torch.from_numpy(X).pin_memory()
        Yp = torch.zeros((c.M, c.N), dtype=torch.float16).pin_memory()
        dX = torch.empty(c.K * ((c.N + 7) // 8 * 8) * 2, dtype=torch.uint8, device="cuda")
        dY = torch.empty(c.M * c.N * 2, dtype=torch.uint8, device="cuda")
        jobs.append((c, W, X, m, Xp, Yp, dX, dY, m.new_workspace(c.N)))
    torch.cuda.synchronize()
    for rep in range(3):
        for (c, W, X, m, Xp, Yp, dX, dY, ws), st in zip(jobs, streams):
            m.spmm_host_async(Xp.numpy(), Yp.numpy(), dX, dY, ws, stream=st)
    for st in streams:
        st.synchronize()
    for c, W, X, m, Xp, Yp, dX, dY, ws in jobs:
        assert m.status(ws) == tl3.OK
        check(oracle_mod, W, X, Yp.numpy(), with_oracle_spmm=False)
        Yb = np.zeros((c.M, c.N), dtype=np.float16)
        m.spmm_host(X, Yb, dX, dY, ws)
        assert np.array_equal(Yb.view(np.uint16), Yp.numpy().view(np.uint16))


def _sampled_check(oracle_mod, W, X, Y, rows):
    Yref, bound = oracle_mod.dense_fp64(W[rows], X)
    err = np.abs(Y[rows].astype(np.float64) - Yref)
    assert np.all(err <= oracle_mod.tolerance(bound))


@pytest.mark.parametrize("config", [2, 3, 4, 5])
def test_full_size_configs_sampled(tl3, oracle_mod, config):
    """The benchmark's shapes in the benchmark's launch configuration; the float64 definition is
    evaluated on a sample of rows (all columns) that covers first, last and straddling row-tiles."""
    import torch
    seen = set()
    for case in wl.config_cases(config):
        key = (case.M, case.K, case.seed)
        if config == 4 and case.M * case.K > 100e6 and case.N != 64:
            continue                                         # the two largest shapes once, at the widest N
        W = case.make_W()
        m = tl3.encode(W)
        if key not in seen:
            seen.add(key)
            assert np.array_equal(m.decode(), W.view(np.uint16))       # bit-exact round trip at full size
        m.upload()
        Xd = torch.from_numpy(case.make_X()).cuda()
        ws = m.new_workspace(case.N)
        Y = m.spmm(Xd, workspace=ws)
        torch.cuda.synchronize()
        assert m.status(ws) == tl3.OK
        Yh = Y.cpu().numpy()
        rng = np.random.default_rng(case.seed)
        rows = np.unique(np.concatenate([np.arange(0, 130), np.arange(case.M - 130, case.M),
                                         rng.integers(0, case.M, 700)]))
        _sampled_check(oracle_mod, W, Xd.cpu().numpy(), Yh, rows)
        assert np.isfinite(Yh.astype(np.float32)).all()
        m.close()
        del Xd, Y, ws
        torch.cuda.empty_cache()


@pytest.mark.parametrize("N", [16, 32])
def test_long_tile_ranges_are_exact_on_small_integers(tl3, oracle_mod, N):
    """20480 x 5120 in the benchmark's launch configuration: 43 tiles per CTA, so the producer reads
    its directory in two batches and every stage, W_r buffer and accumulator barrier wraps many
    times.  With small integers every partial sum is exact in fp32 whatever the order, so ALL rows
    must equal the oracle's format walk and the exact product bit for bit: one dropped or doubled
    weight anywhere shows."""
    rng = np.random.default_rng(2024 + N)
    M, K = 20480, 5120
    W = np.where(rng.random((M, K)) < 0.5, rng.integers(-4, 5, (M, K)), 0).astype(np.float16)
    X = rng.integers(-3, 4, (K, N)).astype(np.float16)
    Y, m = run_gpu(tl3, W, X)
    assert m.last_launch()["ctas"] == 148
    exact = W.astype(np.float64) @ X.astype(np.float64)            # integers below 2^53: exact
    assert np.array_equal(Y.view(np.uint16), exact.astype(np.float16).view(np.uint16))
    assert np.array_equal(Y.view(np.uint16), oracle_mod.spmm(oracle_mod.encode(W), X))


@pytest.mark.parametrize("config,index", [(2, 5), (3, 4), (4, 2), (5, 3)])
def test_full_size_all_rows(tl3, oracle_mod, config, index):
    """One shape of every benchmark configuration, EVERY row against the float64 definition (in row
    blocks to bound memory) and against the oracle's format walk, whose tolerance is tight enough
    to see a single dropped weight."""
    import torch
    case = list(wl.config_cases(config))[index]
    W, X = case.make_W(), case.make_X()
    m = tl3.encode(W)
    m.upload()
    ws = m.new_workspace(case.N)
    Y = m.spmm(torch.from_numpy(X).cuda(), workspace=ws)
    torch.cuda.synchronize()
    assert m.status(ws) == tl3.OK
    Yh = Y.cpu().numpy()
    Yo = oracle_mod.spmm(oracle_mod.encode(W), X).view(np.float16).astype(np.float64)
    for r0 in range(0, case.M, 2048):
        r1 = min(case.M, r0 + 2048)
        Yref, bound = oracle_mod.dense_fp64(W[r0:r1], X)
        y = Yh[r0:r1].astype(np.float64)
        assert np.all(np.abs(y - Yref) <= oracle_mod.tolerance(bound)), (case.name, r0)
        assert np.all(np.abs(y - Yo[r0:r1]) <= 2.0**-9 * np.abs(Yo[r0:r1]) + 1e-4 * bound + 1e-6), (case.name, r0)


def test_decoding_ahead_of_x_changes_no_bit(tl3):
    """The launch option that lets the decode warps start on a block before its X tile has arrived
    only moves a wait: results are bit-identical with it forced on and off."""
    import torch
    outs = []
    case = wl.Case(0, "dbx", 2560, 3072, 24, 9, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    try:
        for setting in (0, -1):
            tl3.set_tuning(decode_before_x=setting)
            Y, _ = run_gpu(tl3, W, X, repeats=2)
            outs.append(Y)
    finally:
        tl3.set_tuning()
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))
    assert tl3.get_tuning()["decode_before_x"] == 4


def test_bind_serves_device_copies_of_the_blob(tl3, oracle_mod):
    """A blob packed on the host and copied over by the caller, and a device-side clone of an
    uploaded blob, give the same bits as the uploaded one; a misaligned pointer is refused."""
    import torch
    case = wl.Case(0, "bind", 1280, 2304, 16, 17, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    m = tl3.encode(W)
    first = m.upload()
    Xd = device_X(X)
    ws = m.new_workspace(case.N)
    Y0 = m.spmm(Xd, workspace=ws).clone()
    check(oracle_mod, W, X, Y0.cpu().numpy())
    packed = torch.from_numpy(m.pack()).cuda()
    clone = first.clone()
    first.zero_()                                               # the old binding must not be read any more
    for blob in (packed, clone):
        m.bind(blob)
        Y = m.spmm(Xd, workspace=ws)
        torch.cuda.synchronize()
        assert m.status(ws) == tl3.OK
        assert torch.equal(Y, Y0)
    assert tl3.lib().tl3_bind(m._h, packed.data_ptr() + 16) == tl3.ERR_INVALID_ARG


def test_row_sharded_matrix_on_one_rank(tl3, oracle_mod):
    """The row-split wrapper with its default per-rank product (the library on the current device);
    with one rank its slab is the whole matrix and no collective runs."""
    import torch
    from paper_2607_08786_b200 import dist
    case = wl.Case(0, "rs", 900, 1024, 16, 5, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    sh = dist.RowShardedMatrix(W)
    Y = sh.matmul(device_X(X))
    torch.cuda.synchronize()
    check(oracle_mod, W, X, Y.cpu().numpy())


def _device_encode_matches(tl3, oracle_mod, W, ld=None):
    import torch
    M, K = W.shape
    buf = torch.zeros((M, ld or K), dtype=torch.float16, device="cuda")
    buf[:, :K] = torch.from_numpy(W)
    m = tl3.Matrix.encode_on_device(buf[:, :K])
    cont = oracle_mod.encode(W)
    for name in tl3.CANONICAL:
        assert np.array_equal(m.canonical(name), getattr(cont, name).ravel()), name
    st = m.stats()
    for key in ("nnz", "n_tc", "n_sf", "n_res", "n_dummy", "n_slots_unused"):
        assert st[key] == cont.stats[key], key
    assert np.array_equal(m.decode(), np.where((W.view(np.uint16) & 0x7FFF) == 0, 0, W.view(np.uint16)))
    return m


@pytest.mark.parametrize("shape,sparsity,kind", [((1024, 1024), 0.5, "bernoulli"), ((640, 896), 0.5, "magnitude"),
                                                 ((1000, 1096), 0.4, "magnitude"), ((130, 260), 0.6, "magnitude"),
                                                 ((384, 512), 0.7, "magnitude"), ((256, 384), 0.0, "bernoulli"),
                                                 ((1, 8), 0.5, "bernoulli"), ((2048, 4096), 0.5, "wanda")])
def test_gpu_encoder_is_byte_identical_to_the_oracle(tl3, oracle_mod, shape, sparsity, kind):
    """The container built by the CUDA encoder (window classification, ordered lists by prefix
    scans, pairing, chain emission, Residual) against the oracle's, array by array and count by
    count, on aligned and ragged shapes and on the dense and sparse side of 50 %."""
    W = wl.Case(0, "ge", shape[0], shape[1], 8, 70 + shape[0], sparsity, kind).make_W()
    _device_encode_matches(tl3, oracle_mod, W)


def test_gpu_encoder_on_hand_built_patterns(tl3, oracle_mod):
    """Dummy points, a chain cut after 255 bytes, cross-row parking, -0.0, a strided source, and the
    product computed from the device-encoded handle."""
    import torch
    from special_cases import clustered_surplus_tile
    rng = np.random.default_rng(3)
    # top half of every tile dense, bottom half empty: every surplus weight is parked in another row
    W = np.zeros((256, 256), dtype=np.float16)
    W[:64] = (rng.standard_normal((64, 256)) * 0.05 + 0.2).astype(np.float16)
    W[128:192] = (rng.standard_normal((64, 256)) * 0.05 + 0.2).astype(np.float16)
    _device_encode_matches(tl3, oracle_mod, W)
    # surplus weights in row 0 only, empty slots spread over the whole tile: long spans of dummy
    # points, and the row's chain runs into the 255-byte limit
    W = (rng.standard_normal((128, 128)) * 0.05 + 0.3).astype(np.float16)
    W[1:, 2::4] = 0
    W[1:, 3::4] = 0
    W[1::2, 1::4] = 0
    m = _device_encode_matches(tl3, oracle_mod, W)
    assert m.stats()["n_dummy"] > 0
    # row 0 dense (64 surplus weights), the other rows exactly 2:4 with one empty slot every 115
    # slots: eight dummy bytes per pair, so the chain of row 0 is cut at 255 bytes and the rest of the
    # row goes to the Residual layer
    W = np.zeros((128, 128), dtype=np.float16)
    base = (rng.standard_normal((128, 128)) * 0.05 + 0.3).astype(np.float16)
    W[0] = base[0]
    W[1:, 0::4] = base[1:, 0::4]
    W[1:, 1::4] = base[1:, 1::4]
    for k in range(70):
        tau = 64 + k * 115
        W[tau // 64, 4 * ((tau % 64) // 2) + (tau & 1)] = 0
    m = _device_encode_matches(tl3, oracle_mod, W)
    assert m.stats()["n_res"] == 32 and m.canonical("chain_len")[0] == 248
    _device_encode_matches(tl3, oracle_mod, clustered_surplus_tile())
    W = wl.Case(0, "neg0", 300, 520, 8, 4, 0.5, "magnitude").make_W()
    W.view(np.uint16)[W == 0] = 0x8000                                  # pruned weights as -0.0
    _device_encode_matches(tl3, oracle_mod, W)
    case = wl.Case(0, "ld", 512, 640, 16, 8, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    m = _device_encode_matches(tl3, oracle_mod, W, ld=648)
    m.upload()
    Y = m.spmm(device_X(X))
    torch.cuda.synchronize()
    check(oracle_mod, W, X, Y.cpu().numpy())


def _gpu_pack_matches(tl3, W):
    """The blob written by the CUDA packer against the host packer's, byte for byte, with the layout
    computed on the GPU (fresh handle) and on the host (second handle)."""
    import torch
    ref = tl3.encode(W)
    want = ref.pack()
    st_ref = ref.stats()
    for host_plan_first in (False, True):
        m = tl3.encode(W)
        if host_plan_first:
            assert m.device_bytes() == want.size
        blob = m.upload_packed_on_device()
        torch.cuda.synchronize()
        got = blob.cpu().numpy()
        assert got.size == want.size
        assert np.array_equal(got, want), f"first difference at byte {int(np.flatnonzero(got != want)[0])}"
        st = m.stats()
        for key in ("device_bytes", "dev_n_sf", "dev_n_res", "dev_n_dummy", "dev_pdd_bytes"):
            assert st[key] == st_ref[key], key
    return m


@pytest.mark.parametrize("shape,sparsity,kind", [((1024, 1024), 0.5, "bernoulli"), ((640, 896), 0.5, "magnitude"),
                                                 ((1000, 1096), 0.4, "magnitude"), ((384, 512), 0.6, "magnitude"),
                                                 ((384, 512), 0.7, "magnitude"), ((256, 384), 0.0, "bernoulli"),
                                                 ((128, 128), 1.0, "bernoulli"), ((2048, 4096), 0.5, "wanda")])
def test_gpu_packer_is_byte_identical_to_the_host_packer(tl3, shape, sparsity, kind):
    W = wl.Case(0, "gp", shape[0], shape[1], 8, 90 + shape[0], sparsity, kind).make_W()
    _gpu_pack_matches(tl3, W)


def test_gpu_packer_on_adversarial_patterns_and_end_to_end(tl3, oracle_mod):
    """Abruptly changing densities (the packer's proportional selection, equal-count chains and the
    cut after three code words), the clustered tile whose chains overflow, and a product computed
    from a matrix that never met the host encoder or the host packer."""
    import torch
    from special_cases import clustered_surplus_tile
    for seed in range(4):
        rng = np.random.default_rng([77, seed])
        M, K = 256, 384
        dens_r = rng.choice([0.0, 0.1, 0.5, 0.9, 1.0], size=M // 32).repeat(32)
        dens_c = rng.choice([0.0, 0.25, 0.5, 0.75, 1.0], size=K // 64).repeat(64)
        p = np.clip(0.5 * (dens_r[:, None] + dens_c[None, :]) + rng.choice([-0.3, 0.0, 0.3]), 0, 1)
        W = np.where(rng.random((M, K)) < p, (rng.standard_normal((M, K)) * 0.05).astype(np.float16), np.float16(0))
        W[(W.view(np.uint16) & 0x7FFF) == 0] = 0
        _gpu_pack_matches(tl3, W)
    _gpu_pack_matches(tl3, clustered_surplus_tile())
    case = wl.Case(0, "gpu_only", 1536, 2048, 16, 61, 0.5, "magnitude")
    W, X = case.make_W(), case.make_X()
    m = tl3.Matrix.encode_on_device(torch.from_numpy(W).cuda())
    m.upload_packed_on_device()
    Y = m.spmm(device_X(X))
    torch.cuda.synchronize()
    check(oracle_mod, W, X, Y.cpu().numpy())


def test_random_shapes_through_every_gpu_route(tl3, oracle_mod):
    """Seeded random shapes, sparsities from dense to 99 %, patchy row densities and padded leading
    dimensions: the CUDA encoder's container and the CUDA packer's blob against the host library's
    (itself pinned to the oracle byte for byte), then the product -- plain, transposed, and with a
    bias and an activation -- against the oracle's fp64 result."""
    import torch
    rng = np.random.default_rng(20260708)
    for it in range(24):
        M = int(rng.integers(1, 12)) * 128 + int(rng.choice([0, 0, 1, 37, 64, 127]))
        K = int(rng.integers(1, 12)) * 128 + int(rng.choice([0, 0, 8, 40, 120]))
        N = int(rng.choice([1, 8, 16, 24, 32, 64]))
        sp = float(rng.choice([0.0, 0.2, 0.4, 0.5, 0.5, 0.6, 0.7, 0.9, 0.99]))
        kind = str(rng.choice(["magnitude", "bernoulli", "row_scaled", "wanda"]))
        case = wl.Case(0, "soak", M, K, N, 500 + it, sp, kind)
        W, X = case.make_W(), case.make_X()
        if it % 3 == 0:
            rows = rng.choice([0.0, 0.3, 1.0], size=(M + 31) // 32).repeat(32)[:M]
            W = np.where(rng.random((M, K)) < rows[:, None], W, np.float16(0))
        tag = f"case {it}: {M}x{K} N={N} sparsity {sp} {kind}"
        ref = tl3.encode(W)
        buf = torch.zeros((M, K + int(rng.choice([0, 8, 24]))), dtype=torch.float16, device="cuda")
        buf[:, :K] = torch.from_numpy(W)
        m = tl3.Matrix.encode_on_device(buf[:, :K])
        for name in tl3.CANONICAL + tl3.COMPACT:
            assert np.array_equal(m.canonical(name), ref.canonical(name)), (tag, name)
        blob = m.upload_packed_on_device()
        torch.cuda.synchronize()
        assert np.array_equal(blob.cpu().numpy(), ref.pack()), tag
        assert m.stats() == ref.stats(), tag
        Xd = device_X(X)
        Y = m.spmm(Xd).cpu().numpy()
        check(oracle_mod, W, X, Y, with_oracle_spmm=False)
        Yt = m.spmm_nt(Xd.t().contiguous()).cpu().numpy()
        assert np.array_equal(Y.view(np.uint16), Yt.T.view(np.uint16)), tag
        bias = (rng.standard_normal(M) * 0.1).astype(np.float16)
        Yb = m.spmm(Xd, bias=torch.from_numpy(bias).cuda(), activation="relu").cpu().numpy().astype(np.float64)
        Yref, bound = oracle_mod.dense_fp64(W, X)
        want = np.maximum(Yref + bias.astype(np.float64)[:, None], 0.0)
        assert np.all(np.abs(Yb - want) <= oracle_mod.tolerance(bound + np.abs(bias.astype(np.float64))[:, None])), tag
        m.close()
        ref.close()


@pytest.mark.parametrize("shape,sparsity,kind", [((1024, 1024), 0.5, "bernoulli"), ((640, 896), 0.4, "magnitude"),
                                                 ((1000, 1096), 0.6, "magnitude"), ((130, 260), 0.9, "magnitude"),
                                                 ((2048, 4096), 0.5, "wanda")])
def test_conversion_that_never_leaves_the_gpu(tl3, oracle_mod, shape, sparsity, kind):
    """Dense W on the device -> container on the device -> packed blob on the device, with no host
    copy of the container: the blob must be the host pipeline's blob byte for byte, the layer counts
    the host encoder's, the product right, and every call that needs the container on the host must
    say so instead of handing out empty arrays."""
    import torch
    case = wl.Case(0, "dev_only", shape[0], shape[1], 16, 130 + shape[0], sparsity, kind)
    W, X = case.make_W(), case.make_X()
    ref = tl3.encode(W)
    want = ref.pack()
    m = tl3.Matrix.encode_on_device(torch.from_numpy(W).cuda(), device_only=True)
    assert m.device_bytes() == want.size
    blob = m.upload_packed_on_device()
    torch.cuda.synchronize()
    assert np.array_equal(blob.cpu().numpy(), want)
    st, st_ref = m.stats(), ref.stats()
    for key in st:
        if key.startswith("canonical_bytes_compact"):
            assert st[key] == -1
        else:
            assert st[key] == st_ref[key], key
    Y = m.spmm(device_X(X))
    torch.cuda.synchronize()
    check(oracle_mod, W, X, Y.cpu().numpy(), with_oracle_spmm=False)
    for call in (m.decode, lambda: m.canonical("tc_vals"), m.serialize, lambda: m.serialize(compact=True), m.pack, m.upload):
        with pytest.raises(tl3.Tl3Error) as e:
            call()
        assert e.value.code == tl3.ERR_UNSUPPORTED
    with pytest.raises(tl3.Tl3Error):                             # the device copy of the container is gone after packing
        m.upload_packed_on_device()
    m.close()
    # a handle that is freed before it was packed releases its device memory (checked where the
    # container is large enough to tell from allocator noise)
    if W.nbytes >= (8 << 20):
        Wd = torch.from_numpy(W).cuda()
        torch.cuda.synchronize()
        free0 = torch.cuda.mem_get_info()[0]
        m2 = tl3.Matrix.encode_on_device(Wd, device_only=True)
        held = free0 - torch.cuda.mem_get_info()[0]
        assert held >= W.nbytes // 2                              # the container is on the device now
        m2.close()
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] >= free0 - (2 << 20)
