"""GPU parity: the CUDA library against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2302_01425_b200 import binding as tk, build, workloads as wl

pytestmark = pytest.mark.gpu

P43 = 4.0 / 3.0


@pytest.fixture(scope="module", autouse=True)
def built():
    build.build()
    tk.load()


def rows_of(n, rows, seed, scale=1.0):
    return wl.normal_rows(rows, n, seed, scale)


@pytest.mark.parametrize("mode", [tk.TK_MASK, tk.TK_TOPK, tk.TK_TOPKMAG])
@pytest.mark.parametrize("p", [2.0, P43])
def test_small_shapes_all_modes(mode, p):
    from parity import run_case
    for n, k, lam, seed in [(1, 1, 1.0, 1), (2, 1, 0.5, 2), (3, 2, 1.0, 3), (5, 5, 1.0, 4),
                            (32, 4, 1.0, 5), (33, 7, 0.3, 6), (64, 2, 0.1, 7), (100, 10, 2.0, 8),
                            (127, 126, 1.0, 9), (129, 1, 1.0, 10), (257, 40, 0.05, 11)]:
        x = rows_of(n, 37, seed)
        g = wl.cotangent_like(x, seed)
        run_case(x, k, p, lam, mode, g, label=f"n={n} k={k} lam={lam} mode={mode} p={p}")


@pytest.mark.parametrize("mode", [tk.TK_MASK, tk.TK_TOPK, tk.TK_TOPKMAG])
@pytest.mark.parametrize("p", [2.0, P43])
def test_multi_tile_rows_with_ragged_tail(mode, p):
    from parity import run_case
    for n, k, lam, seed in [(1000, 5, 0.5, 21), (1500, 150, 1.0, 22), (4096, 512, 1.0, 23),
                            (5000, 77, 0.2, 24), (10007, 1000, 1.0, 25), (16384, 2048, 1.0, 26)]:
        rows = 6 if n > 4096 else 12
        x = rows_of(n, rows, seed)
        g = wl.cotangent_like(x, seed)
        run_case(x, k, p, lam, mode, g, label=f"n={n} k={k} lam={lam} mode={mode} p={p}")


def test_ties_and_signed_zeros():
    from parity import run_case
    x = wl.class_logit_rows(64, 1000, seed=2, scale=3.0)
    g = wl.cotangent_like(x, 2)
    run_case(x, 5, P43, 0.5, tk.TK_TOPK, g, label="class-logit ties")
    y = rows_of(200, 16, 31)
    y[:, 10:20] = 0.0
    y[:, 20:25] = -0.0
    y[:, 30:60] = y[:, 90:120]
    y[:, 130:150] = -y[:, 150:170]
    for mode in (tk.TK_MASK, tk.TK_TOPKMAG):
        for p in (2.0, P43):
            run_case(y, 40, p, 0.7, mode, None, label=f"ties mode={mode} p={p}")
    const = np.full((4, 77), 1.25, np.float32)
    run_case(const, 7, 2.0, 1.0, tk.TK_MASK, None, label="constant row")
    run_case(const, 7, P43, 1.0, tk.TK_TOPKMAG, None, label="constant row mag")


def test_tiny_config_and_figure1():
    from parity import run_case
    for case in wl.tiny_cases():
        x = case.theta()
        g = case.cotangent(x)
        run_case(x, case.k, case.p, case.lam, case.mode, g, label=case.name)


def test_extreme_lambda_and_outliers():
    from parity import run_case
    x = rows_of(96, 20, 41)
    for lam in (1e-6, 1e-3, 50.0, 1e4):
        for p in (2.0, P43):
            run_case(x, 9, p, lam, tk.TK_MASK, None, label=f"lam={lam} p={p}")
            run_case(x, 9, p, lam, tk.TK_TOPKMAG, None, label=f"mag lam={lam} p={p}")
    z = rows_of(300, 10, 42)
    z[:, 0] = 1e6
    z[:, 1] = -1e6
    for p in (2.0, P43):
        run_case(z, 30, p, 1.0, tk.TK_MASK, wl.cotangent_like(z, 42), label=f"outliers p={p}")


def test_argsort_entry_point():
    from oracle import tko
    for mode in (tk.TK_MASK, tk.TK_TOPKMAG):
        for n in (1, 7, 64, 1000, 4099):
            x = rows_of(n, 9, 50 + n)
            if n > 10:
                x[:, 3] = x[:, 9]
                x[:, 5] = -x[:, 6]
            th = torch.from_numpy(x).cuda()
            perm = torch.empty((9, n), dtype=torch.int32, device="cuda")
            srt = torch.empty((9, n), dtype=torch.float32, device="cuda")
            tk.tk_argsort(th, 9, n, mode, perm, srt)
            torch.cuda.synchronize()
            rp, rs = tko.argsort(x, mode)
            assert np.array_equal(perm.cpu().numpy(), rp)
            assert np.array_equal(srt.cpu().numpy().astype(np.float64), rs)


def test_nonfinite_input_sets_status_and_returns():
    x = rows_of(64, 8, 61)
    x[3, 5] = np.nan
    x[5, 0] = np.inf
    th = torch.from_numpy(x).cuda()
    out = torch.empty_like(th)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tk.tk_fwd_ex(th, 8, 64, 4, 2.0, 1.0, tk.TK_MASK, out, status_out=status)
    torch.cuda.synchronize()
    assert int(status.item()) & tk.TK_FLAG_NONFINITE
    from oracle import tko
    ok = [0, 1, 2, 4, 6, 7]
    ref = tko.fwd(x[ok], 4, 2.0, 1.0, tko.MASK)
    assert np.max(np.abs(out.cpu().numpy()[ok] - ref)) <= 1e-5


def test_runs_are_bit_reproducible():
    x = rows_of(2048, 32, 71)
    th = torch.from_numpy(x).cuda()
    a = torch.empty_like(th)
    b = torch.empty_like(th)
    for p in (2.0, P43):
        tk.tk_fwd(th, 32, 2048, 100, p, 1.0, tk.TK_MASK, a)
        tk.tk_fwd(th, 32, 2048, 100, p, 1.0, tk.TK_MASK, b)
        torch.cuda.synchronize()
        assert torch.equal(a, b)


@pytest.mark.parametrize("mode", [tk.TK_MASK, tk.TK_TOPK, tk.TK_TOPKMAG])
@pytest.mark.parametrize("p", [2.0, P43])
def test_rows_held_in_global_memory(mode, p):
    from parity import run_case
    for n, k, lam, rows, seed in [(16385, 1638, 1.0, 3, 81), (20011, 77, 0.3, 2, 82), (32768, 9000, 2.0, 2, 85), (40000, 4000, 1.0, 2, 83),
                                  (70001, 35000, 0.05, 1, 84)]:
        x = rows_of(n, rows, seed)
        if seed == 82:
            x[:, 100:400] = x[:, 5000:5300]        # exact ties across tiles
        g = wl.cotangent_like(x, seed)
        run_case(x, k, p, lam, mode, g, label=f"long n={n} k={k} lam={lam} mode={mode} p={p}")


def test_long_rows_need_a_workspace():
    n = 40000
    th = torch.zeros((1, n), device="cuda")
    out = torch.empty_like(th)
    with pytest.raises(tk.TkError) as e:
        tk.tk_fwd(th, 1, n, 10, 2.0, 1.0, tk.TK_MASK, out)
    assert e.value.status == tk.TK_ERR_WORKSPACE
    need = tk.tk_workspace_bytes(1, n, 10, 2.0, tk.TK_MASK)
    assert need > 0
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(tk.TkError) as e:
        tk.tk_fwd_ex(th, 1, n, 10, 2.0, 1.0, tk.TK_MASK, out, workspace=small)
    assert e.value.status == tk.TK_ERR_WORKSPACE
    # 16384 < n <= 32768: the plain forward pass and the VJP from state run on chip without scratch;
    # a permutation, or a VJP without saved state, still asks for it
    n = 20000
    th = torch.randn((2, n), device="cuda")
    out = torch.empty_like(th)
    st = tk.new_state(2)
    tk.tk_fwd_ex(th, 2, n, 10, 2.0, 1.0, tk.TK_MASK, out, state_out=st)
    tk.tk_vjp(th, th, 2, n, 10, 2.0, 1.0, tk.TK_MASK, out, state=st)
    torch.cuda.synchronize()
    perm = torch.empty((2, n), dtype=torch.int32, device="cuda")
    with pytest.raises(tk.TkError) as e:
        tk.tk_fwd_ex(th, 2, n, 10, 2.0, 1.0, tk.TK_MASK, out, perm_out=perm)
    assert e.value.status == tk.TK_ERR_WORKSPACE
    with pytest.raises(tk.TkError) as e:
        tk.tk_vjp(th, th, 2, n, 10, 2.0, 1.0, tk.TK_MASK, out)
    assert e.value.status == tk.TK_ERR_WORKSPACE


def test_pruning_config_full_size():
    from parity import run_case
    case = wl.pruning_case()
    x = case.theta()
    g = case.cotangent(x)
    res = run_case(x, case.k, case.p, case.lam, case.mode, g, label="pruning 1 x 4194304")
    print("pruning", res)


def test_moe_router_config_full_size():
    """The benchmark's default workload, every variant, every element."""
    from parity import run_case
    for case in wl.moe_router_cases():
        x = case.theta()
        g = case.cotangent(x)
        run_case(x, case.k, case.p, case.lam, case.mode, g, label=case.name)


def test_class_logit_config_full_size():
    from parity import run_case
    case = wl.class_logit_case()
    x = case.theta()
    g = case.cotangent(x)
    run_case(x, case.k, case.p, case.lam, case.mode, g, label=case.name)


def test_expert_choice_config_full_size():
    """32768 x 400, k = 28: the exact path on every element, and 10 Dykstra sweeps against the
    oracle's iteration at the same count."""
    from oracle import tko
    from parity import run_case, TOL
    case = wl.expert_choice_case()
    x = case.theta()
    g = case.cotangent(x)
    run_case(x, case.k, case.p, case.lam, case.mode, g, label=case.name)
    th = torch.from_numpy(x).cuda()
    out = torch.full_like(th, float("nan"))
    tk.tk_fwd_ex(th, case.rows, case.n, case.k, case.p, case.lam, case.mode, out,
                 solver=tk.TK_SOLVER_DYKSTRA, sweeps=10)
    torch.cuda.synchronize()
    ref = tko.dykstra(x, case.k, case.p, case.lam, case.mode, sweeps=10)
    assert float(np.max(np.abs(out.cpu().numpy() - ref))) <= TOL


def test_sweep_configs_full_size_sampled_rows():
    """2^26-element launches as the benchmark times them; the oracle checks a sample of rows."""
    from parity import run_sampled
    for case in wl.shape_sweep_cases():
        if case.n > 4096:
            continue
        x = case.theta()
        g = case.cotangent(x)
        rng = np.random.Generator(np.random.PCG64(case.seed + 77))
        count = max(32, min(4096, (1 << 18) // case.n))
        sample = np.sort(rng.choice(case.rows, size=count, replace=False))
        sample[0], sample[-1] = 0, case.rows - 1          # first and last row of the launch
        res = run_sampled(x, case.k, case.p, case.lam, case.mode, g, sample, label=case.name)
        print(case.name, res)
        del x, g
        torch.cuda.empty_cache()


def test_short_row_kernel_every_batch_count():
    """Rows of up to 256 elements run 1, 2 or the full number of row batches per warp, by row count:
    one case per (lanes per row, batches) pair beyond the single-batch ones the small tests cover."""
    from parity import run_case
    modes = [tk.TK_MASK, tk.TK_TOPK, tk.TK_TOPKMAG]
    cases = [(12, 120001), (24, 60001), (24, 120001), (50, 30001), (50, 120001),
             (100, 15001), (100, 60001), (200, 7501), (200, 30001)]
    for i, (n, rows) in enumerate(cases):
        p = 2.0 if i % 2 == 0 else P43
        lam = (0.1, 1.0, 3.0)[i % 3]
        k = max(1, n // (3 + i % 4))
        x = rows_of(n, rows, 300 + i)
        g = wl.cotangent_like(x, 300 + i)
        run_case(x, k, p, lam, modes[i % 3], g, label=f"n={n} rows={rows} k={k} lam={lam} p={p}")
    # a warp per row (16 or 32 keys per lane), 1, 2 or 4 rows per warp; narrow windows grow the block
    # on one lane, wide ones (large lambda) on the whole warp
    wide = [(300, 15001, 0.05), (400, 4001, 5.0), (512, 8001, 3.0), (512, 15001, 20.0),
            (700, 3001, 4.0), (1024, 7201, 0.2), (1000, 7201, 10.0), (513, 3001, 1.0)]
    for i, (n, rows, lam) in enumerate(wide):
        p = 2.0 if i % 2 == 0 else P43
        k = max(1, n // (2 + i % 5))
        x = rows_of(n, rows, 400 + i)
        g = wl.cotangent_like(x, 400 + i)
        run_case(x, k, p, lam, modes[i % 3], g, label=f"n={n} rows={rows} k={k} lam={lam} p={p}")


def test_sweep_n32768_sampled_rows():
    from parity import run_case
    for case in wl.shape_sweep_cases():
        if case.n != 32768:
            continue
        x = case.theta(rows=3)
        g = case.cotangent(x)
        run_case(x, case.k, case.p, case.lam, case.mode, g, label=case.name)


def test_sweep_n32768_full_launch_sampled_rows():
    """The 2048 x 32768 launches the benchmark times (both p), 32 rows of each checked by the oracle."""
    from parity import run_sampled
    for case in wl.shape_sweep_cases():
        if case.n != 32768:
            continue
        x = case.theta()
        g = case.cotangent(x)
        sample = np.random.Generator(np.random.PCG64(32768)).choice(case.rows, 32, replace=False)
        run_sampled(x, case.k, case.p, case.lam, case.mode, g, np.sort(sample), label=case.name + " full launch")


@pytest.mark.parametrize("p", [2.0, P43])
def test_threshold_form_small_k_and_layout_edges(p):
    """The sort-free default path: k = 1 and k = 2 (the k + 1 largest keys tracked exactly), ties and
    near-ties at the top, row lengths on both sides of every lane layout, row counts that leave the
    last warp partly empty, and the cases where the root sits at the end of its bracket."""
    from parity import run_case
    for n in (17, 31, 32, 33, 63, 64, 65, 127, 128, 129, 255, 256, 257, 511, 512, 513, 1023, 1024, 1025,
              2047, 2048, 2049, 4095, 4096, 4097, 8193, 16385):
        rows = 5 if n > 2048 else 43
        x = rows_of(n, rows, 700 + n)
        g = wl.cotangent_like(x, 700 + n)
        for k, lam in ((1, 1.0), (2, 0.1), (2, 1.0), (max(1, n // 8), 1.0), (n - 1, 0.3), (n, 1.0)):
            if k > n:
                continue
            run_case(x, k, p, lam, tk.TK_MASK, g, check_perm=False, label=f"n={n} k={k} lam={lam} p={p}")
        run_case(x, 2, p, 0.5, tk.TK_TOPK, g, check_perm=False, label=f"topk n={n} k=2 p={p}")
    # ties and near-ties across rank k for k = 1, 2: equal top keys, a runner-up one ulp below,
    # a gap of exactly lambda (no block), a gap a hair below lambda (block with rho = 1 - 1e-7)
    y = rows_of(64, 64, 811)
    y[:, 0] = 3.0; y[:, 1] = 3.0
    y[8:16, 1] = np.nextafter(np.float32(3.0), np.float32(0.0))
    y[16:24, 2] = 3.0
    y[24:32, 1] = 2.5; y[24:32, 2] = 2.0
    y[32:40, 1] = 2.5; y[32:40, 2] = np.nextafter(np.float32(2.0), np.float32(3.0))
    y[40:48, 1] = 2.0
    y[48:56, 1] = np.nextafter(np.float32(2.0), np.float32(3.0))
    gy = wl.cotangent_like(y, 811)
    for k, lam in ((1, 1.0), (2, 0.5), (2, 1.0), (1, 0.5), (3, 0.5)):
        run_case(y, k, p, lam, tk.TK_MASK, gy, check_perm=False, label=f"top ties k={k} lam={lam} p={p}")


@pytest.mark.parametrize("p", [2.0, P43])
def test_dykstra_path_matches_oracle_sweeps(p):
    """Alternating projections with a fixed sweep count: same count in the oracle, <= 1e-5."""
    from oracle import tko
    from parity import rel_err, TOL
    modes = [tk.TK_MASK, tk.TK_TOPK] + ([tk.TK_TOPKMAG] if p == 2.0 else [])
    shapes = [(1, 1, 1.0), (2, 1, 0.5), (7, 3, 1.0), (8, 8, 1.0), (33, 7, 0.3), (64, 2, 0.1), (64, 8, 1.0),
              (200, 20, 1.0), (256, 100, 2.0), (257, 40, 0.5), (1000, 5, 0.5), (4096, 512, 1.0), (5000, 77, 0.2)]
    for mode in modes:
        for n, k, lam in shapes:
            for sweeps in (1, 10, 100):
                if n > 1000 and sweeps == 1:
                    continue
                rows = 9 if n <= 1000 else 3
                x = rows_of(n, rows, 300 + n)
                th = torch.from_numpy(x).cuda()
                out = torch.full_like(th, float("nan"))
                perm = torch.empty((rows, n), dtype=torch.int32, device="cuda")
                tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out, solver=tk.TK_SOLVER_DYKSTRA, sweeps=sweeps,
                             perm_out=perm)
                torch.cuda.synchronize()
                ref = tko.dykstra(x, k, p, lam, mode, sweeps=sweeps)
                got = out.cpu().numpy()
                assert np.isfinite(got).all()
                assert np.array_equal(perm.cpu().numpy(), tko.argsort(x, mode)[0])
                err = rel_err(got, ref).max()
                assert err <= TOL, (mode, n, k, lam, sweeps, err)


@pytest.mark.parametrize("p,mode", [(1.5, tk.TK_MASK), (1.5, tk.TK_TOPK), (1.5, tk.TK_TOPKMAG), (1.2, tk.TK_MASK),
                                    (P43, tk.TK_TOPKMAG)])
def test_dykstra_path_root_solving_pair_step_matches_oracle_sweeps(p, mode):
    """The dual coordinate ascent of App. A.8 for the cases without a closed-form pair step -- any q other
    than 2 and 4, and phi even with p = 4/3: every coordinate solves its two-variable problem by a bracketed
    Newton iteration.  Same sweep count in the oracle (whose pair solve is a bisection), <= 1e-5."""
    from oracle import tko
    from parity import rel_err, TOL
    shapes = [(1, 1, 1.0), (2, 1, 0.5), (7, 3, 1.0), (8, 8, 1.0), (33, 7, 0.3), (64, 8, 1.0), (200, 20, 1.0),
              (257, 40, 0.5), (1000, 5, 0.5), (4096, 512, 1.0)]
    for n, k, lam in shapes:
        for sweeps in (1, 10, 100):
            if n > 1000 and sweeps != 10:
                continue
            rows = 5 if n <= 1000 else 2
            x = rows_of(n, rows, 340 + n)
            th = torch.from_numpy(x).cuda()
            out = torch.full_like(th, float("nan"))
            tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out, solver=tk.TK_SOLVER_DYKSTRA, sweeps=sweeps)
            torch.cuda.synchronize()
            ref = tko.dykstra(x, k, p, lam, mode, sweeps=sweeps)
            got = out.cpu().numpy()
            assert np.isfinite(got).all()
            err = rel_err(got, ref).max()
            assert err <= TOL, (mode, p, n, k, lam, sweeps, err)


@pytest.mark.parametrize("p", [2.0, P43])
def test_dykstra_cluster_rows_match_oracle_sweeps(p):
    """Rows of 16385..131072 elements: the iterate is shared by a thread-block cluster (2, 3, 5 and 8
    blocks here, ragged and full last blocks); same sweep count in the oracle, <= 1e-5; exact
    permutation; a second call on the same workspace gives the same bits."""
    from oracle import tko
    from parity import rel_err, TOL
    modes = [tk.TK_MASK, tk.TK_TOPK] + ([tk.TK_TOPKMAG] if p == 2.0 else [])
    shapes = [(16385, 2048, 1.0, 2, 10), (32768, 4096, 1.0, 3, 100), (40001, 777, 0.3, 2, 10),
              (70000, 7000, 1.0, 1, 10), (131072, 16384, 2.0, 1, 3)]
    for mode in modes:
        for n, k, lam, rows, sweeps in shapes:
            x = rows_of(n, rows, 900 + n % 97)
            x[0, 5] = x[0, 9]                                   # a tie for the stable order
            th = torch.from_numpy(x).cuda()
            ws = torch.empty(tk.tk_workspace_bytes(rows, n, k, p, mode, tk.TK_SOLVER_DYKSTRA), dtype=torch.uint8,
                             device="cuda")
            assert ws.numel() > 0
            outs = []
            for _ in range(2):
                out = torch.full_like(th, float("nan"))
                perm = torch.empty((rows, n), dtype=torch.int32, device="cuda")
                tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out, solver=tk.TK_SOLVER_DYKSTRA, sweeps=sweeps,
                             perm_out=perm, workspace=ws)
                torch.cuda.synchronize()
                outs.append(out.cpu().numpy())
            ref = tko.dykstra(x, k, p, lam, mode, sweeps=sweeps)
            assert np.isfinite(outs[0]).all()
            assert np.array_equal(outs[0], outs[1])
            assert np.array_equal(perm.cpu().numpy(), tko.argsort(x, mode)[0])
            err = rel_err(outs[0], ref).max()
            assert err <= TOL, (mode, n, k, lam, sweeps, err)
    # without a workspace, and beyond eight blocks: refused before any launch
    th = torch.zeros((1, 20000), device="cuda")
    with pytest.raises(tk.TkError) as e:
        tk.tk_fwd_ex(th, 1, 20000, 5, 2.0, 1.0, tk.TK_MASK, torch.empty_like(th), solver=tk.TK_SOLVER_DYKSTRA)
    assert e.value.status == tk.TK_ERR_WORKSPACE
    th = torch.zeros((1, 131073), device="cuda")
    with pytest.raises(tk.TkError) as e:
        tk.tk_fwd_ex(th, 1, 131073, 5, 2.0, 1.0, tk.TK_MASK, torch.empty_like(th), solver=tk.TK_SOLVER_DYKSTRA)
    assert e.value.status == tk.TK_ERR_UNSUPPORTED


def test_smooth_topk_loss_matches_oracle():
    """tk_topk_loss: loss value and gradient (mask - target) against the oracle; rows with no target;
    both row layouts of the reduction pass (warp per row, block per row), vector and scalar access."""
    from oracle import tko
    from parity import rel_err, TOL
    shapes = [(1, 1, 1, 1.0, 2.0), (5, 2, 1, 0.5, 2.0), (64, 10, 3, 1.0, P43), (33, 100, 3, 0.3, 2.0),
              (64, 1000, 3, 0.5, P43), (9, 1001, 5, 0.5, 2.0), (17, 2048, 64, 1.0, 2.0), (5, 5000, 50, 0.2, P43),
              (3, 16384, 2048, 1.0, 2.0), (40, 64, 8, 1.0, 1.5), (3, 4096, 100, 0.7, 1.5)]
    for rows, n, k, lam, p in shapes:
        x = rows_of(n, rows, 500 + n + rows, scale=3.0)
        rng = np.random.default_rng(n)
        tgt = rng.integers(0, n, size=rows).astype(np.int32)
        if rows > 2:
            tgt[1] = -1
            tgt[2] = n
        th = torch.from_numpy(x).cuda()
        loss = torch.full((rows,), float("nan"), device="cuda")
        grad = torch.full_like(th, float("nan"))
        tk.tk_topk_loss(th, torch.from_numpy(tgt).cuda(), rows, n, k, p, lam, loss, grad)
        torch.cuda.synchronize()
        lref, gref = tko.topk_loss(x, tgt, k, p, lam)
        assert rel_err(loss.cpu().numpy(), lref).max() <= TOL, (rows, n, k, lam, p)
        assert rel_err(grad.cpu().numpy(), gref).max() <= TOL, (rows, n, k, lam, p)
    # no target array at all: the value f itself and the mask
    x = rows_of(100, 7, 3)
    th = torch.from_numpy(x).cuda()
    loss = torch.empty((7,), device="cuda")
    grad = torch.empty_like(th)
    tk.tk_topk_loss(th, None, 7, 100, 3, 2.0, 1.0, loss, grad)
    torch.cuda.synchronize()
    lref, gref = tko.topk_loss(x, -np.ones(7), 3, 2.0, 1.0)
    assert rel_err(loss.cpu().numpy(), lref).max() <= TOL
    assert rel_err(grad.cpu().numpy(), tko.fwd(x, 3, 2.0, 1.0, tko.MASK)).max() <= TOL


def test_smooth_topk_loss_class_logit_full_size():
    """8192 x 1000 logits with forced ties, k = 3 and k = 5, p = 4/3 and 2: every row's loss and gradient."""
    from oracle import tko
    from parity import rel_err, TOL
    case = wl.class_logit_case()
    x = case.theta()
    rows, n = x.shape
    tgt = np.random.default_rng(11).integers(0, n, size=rows).astype(np.int32)
    th, tg = torch.from_numpy(x).cuda(), torch.from_numpy(tgt).cuda()
    for k, p in [(3, P43), (5, 2.0)]:
        loss = torch.empty((rows,), device="cuda")
        grad = torch.empty_like(th)
        tk.tk_topk_loss(th, tg, rows, n, k, p, case.lam, loss, grad)
        torch.cuda.synchronize()
        lref, gref = tko.topk_loss(x, tgt, k, p, case.lam)
        assert rel_err(loss.cpu().numpy(), lref).max() <= TOL
        assert rel_err(grad.cpu().numpy(), gref).max() <= TOL


@pytest.mark.parametrize("mode", [tk.TK_MASK, tk.TK_TOPK, tk.TK_TOPKMAG])
def test_straight_through_hard_forward_relaxed_backward(mode):
    """TK_OPT_STRAIGHT_THROUGH: the forward output is the hard operator, bit for bit (ties by index),
    and the VJP from the saved state is the relaxed operator's."""
    from oracle import tko
    from parity import rel_err, TOL
    for n, k, lam, p, rows in [(1, 1, 1.0, 2.0, 3), (8, 3, 0.5, 2.0, 40), (64, 2, 0.1, P43, 33), (400, 28, 1.0, 2.0, 9),
                               (1000, 5, 0.5, P43, 5), (5000, 500, 0.3, 2.0, 3), (20000, 100, 1.0, 2.0, 2)]:
        x = rows_of(n, rows, 700 + n)
        if n >= 8:
            x[0, 1] = x[0, 5] = x[0, 7] = x[0].max() if mode != tk.TK_TOPKMAG else np.abs(x[0]).max()   # ties at the top
        g = wl.cotangent_like(x, 701 + n)
        th, gt = torch.from_numpy(x).cuda(), torch.from_numpy(g).cuda()
        out = torch.full_like(th, float("nan"))
        grad = torch.empty_like(th)
        perm = torch.empty((rows, n), dtype=torch.int32, device="cuda")
        state = tk.new_state(rows)
        wsb = tk.tk_workspace_bytes(rows, n, k, p, mode)
        ws = torch.empty(wsb, dtype=torch.uint8, device="cuda") if wsb else None
        tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out, perm_out=perm, state_out=state, workspace=ws,
                     flags=tk.TK_OPT_STRAIGHT_THROUGH)
        tk.tk_vjp(th, gt, rows, n, k, p, lam, mode, grad, state=state, workspace=ws)
        torch.cuda.synchronize()
        assert np.array_equal(out.cpu().numpy().astype(np.float64), tko.hard(x, k, mode)), (n, k, mode)
        gref = tko.vjp(x, g, k, p, lam, mode)
        assert rel_err(grad.cpu().numpy(), gref).max() <= TOL, (n, k, mode)
    th = torch.zeros((2, 16), device="cuda")
    with pytest.raises(tk.TkError) as e:            # the hard output is read off the permutation
        tk.tk_fwd_ex(th, 2, 16, 3, 2.0, 1.0, mode, torch.empty_like(th), flags=tk.TK_OPT_STRAIGHT_THROUGH)
    assert e.value.status == tk.TK_ERR_INVALID_ARG


@pytest.mark.parametrize("mode", [tk.TK_MASK, tk.TK_TOPK, tk.TK_TOPKMAG])
def test_operator_along_the_slow_axis(mode):
    """tk_fwd_cols / tk_vjp_cols on [n, cols] matrices with a leading dimension: every column against
    the oracle on that column; ragged tiles (neither n nor cols a multiple of 32), ld > cols, the
    padding columns left untouched; the VJP with theta given and with the workspace copy reused."""
    from oracle import tko
    from parity import rel_err, TOL
    for n, cols, ld, k, lam, p in [(1, 1, 1, 1, 1.0, 2.0), (5, 3, 3, 2, 0.5, 2.0), (33, 70, 77, 7, 0.3, P43),
                                   (400, 32, 32, 28, 1.0, 2.0), (64, 1000, 1024, 2, 0.1, 2.0), (1500, 37, 40, 150, 1.0, P43)]:
        if mode == tk.TK_TOPKMAG and p != 2.0 and n > 1000:
            continue
        rng = np.random.default_rng(n * 1000 + cols)
        x = rng.standard_normal((n, ld)).astype(np.float32)
        g = rng.standard_normal((n, ld)).astype(np.float32)
        th, gt = torch.from_numpy(x).cuda(), torch.from_numpy(g).cuda()
        out = torch.full_like(th, -7.0)
        grad = torch.full_like(th, -7.0)
        grad2 = torch.full_like(th, -7.0)
        ws = torch.empty(tk.tk_cols_workspace_bytes(n, cols), dtype=torch.uint8, device="cuda")
        state = tk.new_state(cols)
        tk.tk_fwd_cols(th, n, cols, ld, k, p, lam, mode, out, workspace=ws, state_out=state)
        tk.tk_vjp_cols(None, gt, n, cols, ld, k, p, lam, mode, grad, workspace=ws, state=state)   # reuses theta^T
        tk.tk_vjp_cols(th, gt, n, cols, ld, k, p, lam, mode, grad2, workspace=ws)                 # recomputes
        torch.cuda.synchronize()
        xt, gtt = np.ascontiguousarray(x[:, :cols].T), np.ascontiguousarray(g[:, :cols].T)
        ref = tko.fwd(xt, k, p, lam, mode).T
        gref = tko.vjp(xt, gtt, k, p, lam, mode).T
        o, gr, gr2 = out.cpu().numpy(), grad.cpu().numpy(), grad2.cpu().numpy()
        assert rel_err(o[:, :cols], ref).max() <= TOL, (n, cols, mode)
        assert rel_err(gr[:, :cols], gref).max() <= TOL, (n, cols, mode)
        assert rel_err(gr2[:, :cols], gref).max() <= TOL, (n, cols, mode)
        assert (o[:, cols:] == -7.0).all() and (gr[:, cols:] == -7.0).all()
    th = torch.zeros((8, 8), device="cuda")
    with pytest.raises(tk.TkError) as e:
        tk.tk_fwd_cols(th, 8, 8, 8, 2, 2.0, 1.0, mode, torch.empty_like(th), workspace=None)
    assert e.value.status == tk.TK_ERR_WORKSPACE
    with pytest.raises(tk.TkError) as e:
        tk.tk_fwd_cols(th, 8, 8, 4, 2, 2.0, 1.0, mode, torch.empty_like(th),
                       workspace=torch.empty(4096, dtype=torch.uint8, device="cuda"))
    assert e.value.status == tk.TK_ERR_INVALID_ARG


@pytest.mark.parametrize("p", [2.0, P43])
def test_dykstra_run_to_tolerance_reaches_the_exact_solution(p):
    """tk_opts.tol > 0: the sweeps of a row end once no projection of a sweep moves an entry (p = 2) or a
    dual (p = 4/3) by more than tol; `sweeps` is the cap.  Gated against the exact (pool-adjacent-violators)
    result of the oracle on short rows, where the alternating projections converge quickly; a cap that is
    too small must be reported in the status word, a generous one must not."""
    from oracle import tko
    modes = (tk.TK_MASK, tk.TK_TOPK, tk.TK_TOPKMAG) if p == 2.0 else (tk.TK_MASK, tk.TK_TOPK)
    for n, k, lam, rows in ((8, 3, 0.5, 64), (33, 4, 0.3, 40), (64, 8, 0.5, 130), (300, 6, 0.2, 9), (1000, 5, 0.1, 5)):
        x = rows_of(n, rows, 7100 + n, 1.0)
        th = torch.from_numpy(x).cuda()
        for mode in modes:
            ref = tko.fwd(x, k, p, lam, mode)
            out = torch.full_like(th, float("nan"))
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out, solver=tk.TK_SOLVER_DYKSTRA, sweeps=50000, tol=2e-6,
                         status_out=status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0, (n, mode)
            err = np.abs(out.cpu().numpy().astype(np.float64) - ref) / np.maximum(1.0, np.abs(ref))
            assert err.max() <= 1e-3, f"n={n} mode={mode} p={p}: {err.max()}"
            # the same rows with a cap of two sweeps: rows that pool more than a pair cannot have settled
            status.zero_()
            tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out, solver=tk.TK_SOLVER_DYKSTRA, sweeps=2, tol=2e-6,
                         status_out=status)
            torch.cuda.synchronize()
            assert int(status.item()) & tk.TK_FLAG_NOT_CONVERGED, (n, mode)
            # tol = 0 keeps the fixed count, whatever happens in the sweeps: no flag
            status.zero_()
            tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out, solver=tk.TK_SOLVER_DYKSTRA, sweeps=2, status_out=status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
    big = torch.zeros(2, 20000, device="cuda")
    with pytest.raises(tk.TkError) as e:
        tk.tk_fwd_ex(big, 2, 20000, 5, 2.0, 1.0, tk.TK_MASK, torch.empty_like(big), solver=tk.TK_SOLVER_DYKSTRA,
                     tol=1e-6, workspace=torch.empty(tk.tk_workspace_bytes(2, 20000, 5, 2.0, 0, tk.TK_SOLVER_DYKSTRA),
                                                     dtype=torch.uint8, device="cuda"))
    assert e.value.status == tk.TK_ERR_UNSUPPORTED


def test_dykstra_default_sweeps_and_limits():
    from oracle import tko
    x = rows_of(64, 16, 77)
    th = torch.from_numpy(x).cuda()
    out = torch.empty_like(th)
    tk.tk_fwd_ex(th, 16, 64, 2, 2.0, 0.3, tk.TK_MASK, out, solver=tk.TK_SOLVER_DYKSTRA)   # sweeps = 0 -> 100
    torch.cuda.synchronize()
    ref = tko.dykstra(x, 2, 2.0, 0.3, tko.MASK, sweeps=100)
    assert np.max(np.abs(out.cpu().numpy() - ref)) <= 1e-5
    exact = tko.fwd(x, 2, 2.0, 0.3, tko.MASK)
    assert np.max(np.abs(out.cpu().numpy() - exact)) <= 1e-4       # small blocks: 100 sweeps reach PAV
    big = torch.zeros(2, 20000, device="cuda")
    ws = torch.empty(tk.tk_workspace_bytes(2, 20000, 5, P43, tk.TK_TOPKMAG, tk.TK_SOLVER_DYKSTRA), dtype=torch.uint8, device="cuda")
    with pytest.raises(tk.TkError) as e:          # phi even with p = 4/3: rows of one thread block only
        tk.tk_fwd_ex(big, 2, 20000, 5, P43, 0.3, tk.TK_TOPKMAG, torch.empty_like(big), solver=tk.TK_SOLVER_DYKSTRA,
                     workspace=ws)
    assert e.value.status == tk.TK_ERR_UNSUPPORTED
    with pytest.raises(tk.TkError) as e:
        tk.tk_fwd_ex(th, 16, 64, 2, 2.0, 0.3, tk.TK_MASK, out, solver=tk.TK_SOLVER_DYKSTRA,
                     state_out=tk.new_state(16))
    assert e.value.status == tk.TK_ERR_UNSUPPORTED


@pytest.mark.parametrize("mode", [tk.TK_MASK, tk.TK_TOPK, tk.TK_TOPKMAG])
@pytest.mark.parametrize("p", [2.0, P43])
def test_sort_free_solver_matches_oracle(mode, p):
    """TK_SOLVER_THRESHOLD: same values, same pooled block, and a row state the VJP accepts."""
    from parity import run_case
    shapes = [(1, 1, 1.0, 1), (2, 1, 0.5, 2), (5, 5, 1.0, 4), (33, 7, 0.3, 6), (64, 2, 0.1, 7), (64, 8, 1.0, 7),
              (257, 40, 0.05, 11), (1000, 5, 0.5, 21), (1500, 150, 1.0, 22), (4096, 512, 1.0, 23),
              (5000, 77, 0.2, 24), (10007, 1000, 1.0, 25), (16384, 2048, 1.0, 26), (4096, 400, 1e-3, 27)]
    for n, k, lam, seed in shapes:
        rows = 4 if n > 4096 else 11
        x = rows_of(n, rows, seed, 0.02 if lam == 1e-3 else 1.0)
        g = wl.cotangent_like(x, seed)
        run_case(x, k, p, lam, mode, g, solver=tk.TK_SOLVER_THRESHOLD,
                 label=f"sort-free n={n} k={k} lam={lam} mode={mode} p={p}")


def test_sort_free_solver_ties_outliers_and_limits():
    from parity import run_case
    x = wl.class_logit_rows(64, 1000, seed=2, scale=3.0)
    run_case(x, 5, P43, 0.5, tk.TK_TOPK, wl.cotangent_like(x, 2), solver=tk.TK_SOLVER_THRESHOLD, label="ties")
    y = rows_of(200, 16, 31)
    y[:, 10:20] = 0.0
    y[:, 20:25] = -0.0
    y[:, 30:60] = y[:, 90:120]
    y[:, 130:150] = -y[:, 150:170]
    for mode in (tk.TK_MASK, tk.TK_TOPKMAG):
        for p in (2.0, P43):
            run_case(y, 40, p, 0.7, mode, None, solver=tk.TK_SOLVER_THRESHOLD, label=f"ties mode={mode} p={p}")
    const = np.full((4, 77), 1.25, np.float32)
    run_case(const, 7, 2.0, 1.0, tk.TK_MASK, None, solver=tk.TK_SOLVER_THRESHOLD, label="constant row")
    w = rows_of(96, 20, 41)
    for p in (2.0, P43):
        run_case(w, 9, p, 1e-6, tk.TK_MASK, None, solver=tk.TK_SOLVER_THRESHOLD, label=f"lam=1e-6 p={p}")
        run_case(w, 9, p, 1e-6, tk.TK_TOPKMAG, None, solver=tk.TK_SOLVER_THRESHOLD, label=f"mag lam=1e-6 p={p}")
    z = rows_of(300, 10, 42)
    z[:, 0] = 1e6
    z[:, 1] = -1e6
    # (lambda = 1e-6 next to keys of 1e6 is left out: there the fp64 oracle's own rho(s - (s - lambda))
    # is off by eps |s| / lambda = 2e-4, more than the tolerance; the kernels return exactly 1)
    for lam in (1e-3, 1.0, 50.0, 1e4):
        for p in (2.0, P43):
            run_case(z, 30, p, lam, tk.TK_MASK, None, solver=tk.TK_SOLVER_THRESHOLD, label=f"outliers lam={lam}")
            run_case(z, 30, p, lam, tk.TK_TOPKMAG, None, solver=tk.TK_SOLVER_THRESHOLD, label=f"mag lam={lam}")
    th = torch.from_numpy(z).cuda()
    with pytest.raises(tk.TkError) as e:
        tk.tk_fwd_ex(th, 10, 300, 30, 2.0, 1.0, tk.TK_MASK, torch.empty_like(th), solver=tk.TK_SOLVER_THRESHOLD,
                     perm_out=torch.empty((10, 300), dtype=torch.int32, device="cuda"))
    assert e.value.status == tk.TK_ERR_UNSUPPORTED


@pytest.mark.parametrize("mode", [tk.TK_MASK, tk.TK_TOPK, tk.TK_TOPKMAG])
@pytest.mark.parametrize("p", [1.5, 1.2, 1.1])
def test_general_p_matches_oracle(mode, p):
    """p other than 2 and 4/3 (q = 3, 6, 11): forward pass by the sort-free solver, VJP from state."""
    from parity import run_case
    # the oracle's block solve for these p is a bisection per block member: small row counts
    for n, k, lam, rows, seed in [(64, 2, 0.3, 96, 501), (300, 40, 1.0, 6, 502), (1000, 5, 0.5, 3, 503),
                                  (5000, 700, 2.0, 1, 504)]:
        x = rows_of(n, rows, seed)
        g = wl.cotangent_like(x, seed)
        res = run_case(x, k, p, lam, mode, g, label=f"p={p} n={n} k={k} lam={lam} mode={mode}",
                       solver=tk.TK_SOLVER_THRESHOLD)
        assert "vjp_state_max_rel" in res
    if mode == tk.TK_TOPKMAG:      # phi even: the sort-free solver at every length, VJP from state only
        return
    # rows of up to 128 elements take the sorting kernel with a per-row Newton iteration (solver AUTO):
    # forward, VJP from state and recomputing VJP
    for n, k, lam, rows, seed in [(8, 3, 0.5, 200, 511), (16, 2, 1.0, 130, 512), (64, 2, 0.3, 300, 513),
                                  (64, 20, 3.0, 64, 514), (100, 10, 1.0, 40, 515), (128, 64, 10.0, 33, 516)]:
        x = rows_of(n, rows, seed)
        g = wl.cotangent_like(x, seed)
        res = run_case(x, k, p, lam, mode, g, label=f"sorted p={p} n={n} k={k} lam={lam} mode={mode}")
        assert "vjp_state_max_rel" in res and "vjp_recompute_max_rel" in res


@pytest.mark.parametrize("mode", [tk.TK_MASK, tk.TK_TOPK, tk.TK_TOPKMAG])
def test_general_p_vjp_without_saved_state_recomputes_the_forward_pass(mode):
    """tk_vjp for a general p on rows the sorting kernel does not take, with no saved row state: the forward
    pass runs again (row state into the workspace) and the result is the VJP from state, which is the
    oracle's."""
    from oracle import tko
    p = 1.5
    for n, k, lam, rows in ((300, 40, 1.0, 6), (1000, 5, 0.5, 3), (100, 10, 0.7, 40)):
        if n <= 128 and mode != tk.TK_TOPKMAG:
            continue                                   # those rows have their own recomputing kernel
        x = rows_of(n, rows, 560 + n)
        g = wl.cotangent_like(x, 560 + n)
        th, gt = torch.from_numpy(x).cuda(), torch.from_numpy(g).cuda()
        need = tk.tk_workspace_bytes(rows, n, k, p, mode)
        assert need >= rows * 16
        ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        grad = torch.full_like(th, float("nan"))
        tk.tk_vjp(th, gt, rows, n, k, p, lam, mode, grad, workspace=ws)
        st = tk.new_state(rows)
        out, grad2 = torch.empty_like(th), torch.empty_like(th)
        tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out, state_out=st)
        tk.tk_vjp(th, gt, rows, n, k, p, lam, mode, grad2, state=st)
        torch.cuda.synchronize()
        assert torch.equal(grad, grad2), (n, mode)
        ref = tko.vjp(x, g, k, p, lam, mode)
        a = grad.cpu().numpy().astype(np.float64)
        # rows whose block edge is a near-tie are handled by the full harness elsewhere; here the bulk must agree
        err = np.abs(a - ref) / np.maximum(1.0, np.abs(ref))
        assert np.median(err.max(axis=1)) <= 1e-5, (n, mode, err.max())


def test_vjp_without_saved_state_uses_the_sort_free_forward_when_given_room():
    """tk_vjp with no saved row state but a workspace of rows * 16 bytes: the threshold-form forward pass runs
    again and the VJP is the one from state, bit for bit; without the workspace the sorting kernels recompute,
    and both agree to rounding."""
    for n, k, rows, mode, p in ((64, 8, 500, tk.TK_MASK, 2.0), (1000, 5, 40, tk.TK_TOPK, P43),
                                (4096, 512, 9, tk.TK_TOPKMAG, 2.0), (20000, 300, 3, tk.TK_MASK, P43)):
        x = rows_of(n, rows, 590 + n)
        g = wl.cotangent_like(x, 590 + n)
        th, gt = torch.from_numpy(x).cuda(), torch.from_numpy(g).cuda()
        ws = torch.empty(((rows * 16 + 255) // 256) * 256, dtype=torch.uint8, device="cuda")
        fast, ref, slow = (torch.full_like(th, float("nan")) for _ in range(3))
        tk.tk_vjp(th, gt, rows, n, k, p, 0.7, mode, fast, workspace=ws)
        st = tk.new_state(rows)
        out = torch.empty_like(th)
        tk.tk_fwd_ex(th, rows, n, k, p, 0.7, mode, out, state_out=st)
        tk.tk_vjp(th, gt, rows, n, k, p, 0.7, mode, ref, state=st)
        torch.cuda.synchronize()
        assert torch.equal(fast, ref), (n, mode)
        if n <= 16384:
            tk.tk_vjp(th, gt, rows, n, k, p, 0.7, mode, slow)
            torch.cuda.synchronize()
            d = ((slow - ref).abs() / ref.abs().clamp(min=1.0))
            # rows whose block edge is a near-tie may differ between the two solves: the bulk must agree
            assert float(d.max(dim=1).values.median()) <= 1e-5, (n, mode)


def test_general_p_limits():
    th = torch.randn((4, 64), device="cuda")
    out = torch.empty_like(th)
    tk.tk_fwd(th, 4, 64, 2, 1.5, 1.0, tk.TK_MASK, out)                     # solver AUTO, short row: the sorting kernel
    ref = torch.empty_like(th)
    tk.tk_fwd_ex(th, 4, 64, 2, 1.5, 1.0, tk.TK_MASK, ref, solver=tk.TK_SOLVER_THRESHOLD)
    torch.cuda.synchronize()
    assert float((out - ref).abs().max()) <= 1e-6
    th2 = torch.randn((4, 300), device="cuda")
    out2, ref2 = torch.empty_like(th2), torch.empty_like(th2)
    tk.tk_fwd(th2, 4, 300, 9, 1.5, 1.0, tk.TK_MASK, out2)                  # longer row: routed to the sort-free solver
    tk.tk_fwd_ex(th2, 4, 300, 9, 1.5, 1.0, tk.TK_MASK, ref2, solver=tk.TK_SOLVER_THRESHOLD)
    torch.cuda.synchronize()
    assert torch.equal(out2, ref2)
    g2 = torch.randn_like(th2)
    with pytest.raises(tk.TkError) as e:
        tk.tk_vjp(th2, g2, 4, 300, 9, 1.5, 1.0, tk.TK_MASK, out2)          # no saved state on a row of more than 128:
    assert e.value.status == tk.TK_ERR_WORKSPACE                           # the forward pass runs again and needs room
    for kwargs in ({"solver": tk.TK_SOLVER_PAV},
                   {"perm_out": torch.empty((4, 64), dtype=torch.int32, device="cuda")}):
        with pytest.raises(tk.TkError) as e:
            tk.tk_fwd_ex(th, 4, 64, 2, 1.5, 1.0, tk.TK_MASK, out, **kwargs)
        assert e.value.status == tk.TK_ERR_UNSUPPORTED
    with pytest.raises(tk.TkError) as e:                                   # q < 2
        tk.tk_fwd(th, 4, 64, 2, 3.0, 1.0, tk.TK_MASK, out)
    assert e.value.status == tk.TK_ERR_UNSUPPORTED


@pytest.mark.parametrize("mode", [tk.TK_MASK, tk.TK_TOPK, tk.TK_TOPKMAG])
def test_forward_pass_between_p_1_5_and_2(mode):
    """1.5 < p < 2 (2 < q < 3): the forward pass (and the smooth top-k loss) is served, derivatives are
    refused (rho'' is unbounded at 0 there)."""
    from oracle import tko
    for p, n, k, lam, rows in ((1.8, 64, 5, 0.5, 40), (1.6, 300, 30, 1.0, 8), (1.9, 1000, 100, 2.0, 4)):
        x = rows_of(n, rows, 520 + n)
        th = torch.from_numpy(x).cuda()
        out = torch.full_like(th, float("nan"))
        st = tk.new_state(rows)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out, state_out=st, status_out=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        ref = tko.fwd(x, k, p, lam, mode)
        err = np.abs(out.cpu().numpy() - ref) / np.maximum(1.0, np.abs(ref))
        assert err.max() <= 1e-5, (p, n, err.max())
        g = torch.randn_like(th)
        for call in (lambda: tk.tk_vjp(th, g, rows, n, k, p, lam, mode, out, state=st),
                     lambda: tk.tk_jvp(th, g, rows, n, k, p, lam, mode, out, state=st)):
            with pytest.raises(tk.TkError) as e:
                call()
            assert e.value.status == tk.TK_ERR_UNSUPPORTED


@pytest.mark.parametrize("mode", [tk.TK_MASK, tk.TK_TOPK, tk.TK_TOPKMAG])
@pytest.mark.parametrize("p", [2.0, P43])
def test_jvp_matches_oracle_and_is_the_adjoint_of_the_vjp(mode, p):
    from oracle import tko
    from parity import rel_err, TOL
    # element by element against the oracle's Jacobian on small rows
    for n, k, lam, rows, seed in [(8, 3, 0.7, 40, 601), (33, 7, 0.3, 12, 602), (100, 10, 2.0, 6, 603),
                                  (300, 40, 1.0, 3, 604), (1500, 150, 1.0, 1, 605)]:
        x = rows_of(n, rows, seed)
        v = wl.cotangent_like(x, seed)
        th, vt = torch.from_numpy(x).cuda(), torch.from_numpy(v).cuda()
        out, st, jv = torch.empty_like(th), tk.new_state(rows), torch.empty_like(th)
        tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out, state_out=st)
        tk.tk_jvp(th, vt, rows, n, k, p, lam, mode, jv, state=st)
        torch.cuda.synchronize()
        ref = tko.jvp(x, v, k, p, lam, mode)
        assert float(rel_err(jv.cpu().numpy(), ref).max()) <= 5 * TOL, (n, k, lam)   # n-term sums of 1e-5 entries
    # <g, J v> = <J^T g, v> at a size the oracle's n^2 assembly cannot reach
    rows, n, k, lam = 4096, 400, 28, 1.0
    x = rows_of(n, rows, 610)
    th = torch.from_numpy(x).cuda()
    g = torch.from_numpy(wl.cotangent_like(x, 611)).cuda()
    v = torch.from_numpy(wl.cotangent_like(x, 612)).cuda()
    out, st = torch.empty_like(th), tk.new_state(rows)
    jv, jtg = torch.empty_like(th), torch.empty_like(th)
    tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out, state_out=st)
    tk.tk_jvp(th, v, rows, n, k, p, lam, mode, jv, state=st)
    tk.tk_vjp(th, g, rows, n, k, p, lam, mode, jtg, state=st)
    torch.cuda.synchronize()
    lhs = (g.double() * jv.double()).sum(dim=1)
    rhs = (jtg.double() * v.double()).sum(dim=1)
    scale = (g.double().abs() * jv.double().abs()).sum(dim=1) + 1.0
    assert float(((lhs - rhs).abs() / scale).max()) <= 1e-5
    with pytest.raises(tk.TkError) as e:
        tk.tk_jvp(th, v, rows, n, k, p, lam, mode, jv, state=None)
    assert e.value.status == tk.TK_ERR_UNSUPPORTED


def test_randomised_shapes_modes_and_lambdas():
    """A seeded sweep over row lengths around every kernel boundary, k anywhere in 1..n, lambda from
    0.05 to 100, all modes, exact ties and exact zeros: every case through the full parity harness."""
    from parity import run_case
    rng = np.random.Generator(np.random.PCG64(2024))
    lengths = [1, 2, 3, 5, 8, 9, 13, 16, 17, 31, 32, 33, 64, 65, 100, 128, 129, 200, 256, 257, 300, 400, 512,
               513, 700, 1000, 1024, 1025, 1500, 2048, 2049, 3000, 4096, 5000, 8192, 10000, 16384, 16385,
               20000, 32768]
    for it in range(160):
        n = int(rng.choice(lengths))
        k = int(rng.integers(1, n + 1))
        if rng.random() < 0.5:
            k = max(1, min(n, int(n * rng.choice([0.01, 0.1, 0.25, 0.5, 0.9]))))
        lam = float(rng.choice([0.05, 0.1, 0.3, 1.0, 3.0, 10.0, 100.0]))
        p = float(rng.choice([2.0, P43]))
        mode = int(rng.integers(0, 3))
        rows = int(rng.choice([1, 3, 7, 37])) if n > 2048 else int(rng.choice([1, 5, 37, 130, 1000]))
        scale = float(rng.choice([0.5, 1.0, 1.0, 2.0]))
        x = wl.normal_rows(rows, n, 9000 + it, scale)
        ties = rng.random() < 0.2 and n >= 8
        zeros = rng.random() < 0.1
        if ties:
            x[:, : n // 4] = x[:, n // 2: n // 2 + n // 4]
        if zeros:
            x[:, ::3] = 0.0
        g = wl.cotangent_like(x, 9000 + it)
        run_case(x, k, p, lam, mode, g,
                 label=f"it={it} n={n} k={k} lam={lam} p={p:.3f} mode={mode} rows={rows} ties={ties} zeros={zeros}")


def test_unaligned_base_pointers_take_the_scalar_path_and_agree():
    """theta / cotangent / outputs that start 4 or 12 bytes off a 16-byte boundary cannot use 128-bit
    accesses; the scalar path must give the same results (the summation order of the VJP's block
    sums may differ: one ulp)."""
    for n, k in [(8, 2), (64, 5), (300, 30), (512, 64), (1024, 100), (4096, 512), (16384, 999), (32768, 100)]:
        rows = 33 if n <= 1024 else 3
        for mode, p in [(tk.TK_MASK, 2.0), (tk.TK_TOPK, P43), (tk.TK_TOPKMAG, 2.0)]:
            base = torch.randn(rows * n, device="cuda")
            gbase = torch.randn(rows * n, device="cuda")
            got = []
            for off in (0, 1, 3):
                bufs = [torch.empty(rows * n + 4, device="cuda") for _ in range(5)]
                x, g, o, d, d2 = [b[off:off + rows * n] for b in bufs]
                x.copy_(base); g.copy_(gbase)
                st = tk.new_state(rows)
                tk.tk_fwd_ex(x, rows, n, k, p, 0.7, mode, o, state_out=st)
                tk.tk_vjp(x, g, rows, n, k, p, 0.7, mode, d, state=st)
                if n <= 16384:
                    tk.tk_vjp(x, g, rows, n, k, p, 0.7, mode, d2)
                else:
                    d2.zero_()
                torch.cuda.synchronize()
                got.append((o.clone(), d.clone(), d2.clone()))
            for o, d, d2 in got[1:]:
                assert torch.equal(o, got[0][0]), (n, mode)
                for a, b in ((d, got[0][1]), (d2, got[0][2])):
                    assert float(((a - b).abs() / b.abs().clamp(min=1.0)).max()) <= 1e-6, (n, mode)


@pytest.mark.parametrize("p", [2.0, P43])
def test_general_sorted_w_matches_oracle(p):
    """tk_fwd_w / tk_vjp_w (relaxed linear maximisation over the permutahedron of any sorted w) against
    the oracle's stack PAV: w = 1_k (must also equal the top-k mask path), a ramp, a three-level w,
    the relaxed rank and the relaxed sort.  The VJP jumps where two blocks merge, so elements whose
    pooled block changes under a 1e-6 relative perturbation of theta in the oracle are left out of it."""
    from oracle import tko
    TOL = 1e-5

    def rel(a, b):
        return np.abs(a - b) / np.maximum(1.0, np.abs(b))

    def stable_elements(x, w, lam):
        """[rows, n] mask of the elements whose pooled block (as a set of ranks) is the same for theta and
        for two perturbed copies of it: Prop. 7's Jacobian of an element involves its own block only."""
        def blocks_by_index(det):
            lo = np.empty_like(det["block_lo"]); hi = np.empty_like(det["block_hi"])
            np.put_along_axis(lo, det["perm"].astype(np.int64), det["block_lo"], axis=1)
            np.put_along_axis(hi, det["perm"].astype(np.int64), det["block_hi"], axis=1)
            return lo, hi
        _, d0 = tko.fwd_w(x, w, p, lam, details=True)
        lo0, hi0 = blocks_by_index(d0)
        ok = np.ones(x.shape, bool)
        rng = np.random.Generator(np.random.PCG64(5))
        for _ in range(2):
            xq = (x.astype(np.float64) * (1.0 + 1e-6 * rng.standard_normal(x.shape)) + 1e-6 * rng.standard_normal(x.shape)).astype(np.float32)
            _, d1 = tko.fwd_w(xq, w, p, lam, details=True)
            lo1, hi1 = blocks_by_index(d1)
            ok &= (lo0 == lo1) & (hi0 == hi1)
        return ok

    def run(x, w, lam, label):
        rows, n = x.shape
        th = torch.from_numpy(np.ascontiguousarray(x)).cuda()
        wt = torch.from_numpy(np.ascontiguousarray(w, np.float32)).cuda()
        w64 = np.asarray(wt.cpu().numpy(), np.float64)             # the oracle sees the fp32 values the GPU sees
        out = torch.full((rows, n), float("nan"), device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        tk.tk_fwd_w(th, wt, rows, n, p, lam, out, status_out=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        ref = tko.fwd_w(x, w64, p, lam)
        e = rel(out.cpu().numpy().astype(np.float64), ref)
        assert e.max() <= TOL, f"{label}: forward {e.max()}"
        g = wl.cotangent_like(x, 77)
        gt = torch.from_numpy(g).cuda()
        grad = torch.full((rows, n), float("nan"), device="cuda")
        gw = torch.full((rows, n), float("nan"), device="cuda")
        tk.tk_vjp_w(th, wt, gt, rows, n, p, lam, grad, grad_w=gw)
        torch.cuda.synchronize()
        gref, gwref = tko.vjp_w(x, w64, g, p, lam, with_w=True)
        ok = stable_elements(x, w64, lam)
        assert ok.mean() >= 0.5, f"{label}: only {ok.mean():.2f} of the elements away from a merge"
        eg = rel(grad.cpu().numpy().astype(np.float64), gref)[ok]
        assert np.isfinite(grad.cpu().numpy()).all()
        assert eg.max() <= TOL, f"{label}: vjp {eg.max()}"
        # the cotangent pulled back to w is indexed by sorted rank: the same filter, through the oracle's permutation
        _, det = tko.fwd_w(x, w64, p, lam, details=True)
        ok_rank = np.take_along_axis(ok, det["perm"].astype(np.int64), axis=1)
        assert np.isfinite(gw.cpu().numpy()).all()
        ew = rel(gw.cpu().numpy().astype(np.float64), gwref)[ok_rank]
        assert ew.max() <= TOL, f"{label}: cotangent in w {ew.max()}"
        return out

    for n, rows in ((5, 33), (64, 40), (100, 17), (1000, 9), (2048, 5)):
        x = rows_of(n, rows, 900 + n, 1.5)
        k = max(1, n // 5)
        for lam in (0.3, 2.0):
            ones_k = np.r_[np.ones(k), np.zeros(n - k)].astype(np.float32)
            o = run(x, ones_k, lam, f"1_k n={n} lam={lam}")
            mask = torch.empty_like(o)
            tk.tk_fwd(torch.from_numpy(x).cuda(), rows, n, k, p, lam, tk.TK_MASK, mask)
            torch.cuda.synchronize()
            assert float((o - mask).abs().max()) <= 2e-5, f"n={n}: general-w path differs from the mask path"
            run(x, np.arange(n, 0, -1, dtype=np.float32) / n, lam, f"ramp n={n} lam={lam}")
            levels = np.r_[np.full(n // 3, 2.0), np.full(n // 3, 0.5), np.full(n - 2 * (n // 3), -0.25)].astype(np.float32)
            run(x, levels, lam, f"levels n={n} lam={lam}")
        # relaxed rank of x: theta = -x, w = (n, .., 1); relaxed sort: theta = (n, .., 1), w = x sorted, per row
        rho_v = np.arange(n, 0, -1, dtype=np.float32)
        run(-x, rho_v, 0.5 * n, f"rank n={n}")
        run(-x, rho_v, 1.0, f"rank small lambda n={n}")
        ws = -np.sort(-x, axis=1)
        run(np.tile(rho_v, (rows, 1)), ws, 1.0, f"sort n={n}")
    # limits of the entry points
    th = torch.zeros(4, 4096, device="cuda"); wt = torch.zeros(4096, device="cuda"); o = torch.empty_like(th)
    with pytest.raises(tk.TkError) as e:
        tk.tk_fwd_w(th, wt, 4, 4096, p, 1.0, o)
    assert e.value.status == tk.TK_ERR_UNSUPPORTED
    with pytest.raises(tk.TkError) as e:
        tk.tk_fwd_w(th, wt, 4, 1024, 1.5, 1.0, o)
    assert e.value.status == tk.TK_ERR_UNSUPPORTED

