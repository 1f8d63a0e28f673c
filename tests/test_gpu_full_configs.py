"""The benchmark configurations at full size, in the launch configuration that
bench.py times (tensor-core GEMMs, overlapped anchor refresh, olsgd_run)."""
import json
import os

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import synth_inputs as si
from oracle import models, olsgd, runner, sampling
from conftest import GOLDEN
from helpers import max_rel_err, state_err, to_dev

TOL_BF16_LOSS = 2e-2      # acceptance bar of the bf16-GEMM paths, relative, on the loss


def _gpu(name, iters, table=None, seed=0):
    from paper_2002_09539_b200 import OverlapLocalSGD
    c = si.CONFIGS[name]
    if c["kind"] == "linreg":
        X, y, _ = si.linreg_data(seed, c["m"], c["n"], c["dims"][0])
    else:
        X, y = si.mixture_data(seed, c["m"], c["n"], c["dims"][0], table)
    x0 = si.model_init(seed, c["kind"], c["dims"])
    opt = OverlapLocalSGD(c["kind"], m=c["m"], tau=c["tau"], gamma=c["gamma"], alpha=c["alpha"],
                          beta=c["beta"], mu=c["mu"], batch=c["batch"], seed=seed, dims=c["dims"],
                          gemm_bf16=c["gemm_bf16"], x0=x0, X=to_dev(X), y=to_dev(y))
    loss = torch.zeros((iters, c["m"]), device="cuda")
    opt.run(iters, loss)
    return c, X, y, x0, opt, loss.cpu().numpy()


def _oracle(c, X, y, x0, iters, seed=0):
    return runner.run_model(c["kind"], c["dims"], X, y, x0, m=c["m"], tau=c["tau"],
                            batch=c["batch"], gamma=c["gamma"], alpha=c["alpha"], beta=c["beta"],
                            mu=c["mu"], seed=seed, iters=iters)


def test_config2_full_length():
    c, X, y, x0, opt, lg = _gpu("c2", 500)
    st, lo, _ = _oracle(c, X, y, x0, 500)
    err = state_err(opt, st)
    assert err <= 5e-5, err                       # the 1e-5 bar is stated at 100 iterations
    assert np.abs(lg - lo).max() <= 1e-4 * np.abs(lo).max()
    F_gpu = models.full_objective("softmax", c["dims"], opt.get_params(-4), X, y)
    F_or = models.full_objective("softmax", c["dims"], st.mean_model(), X, y)
    assert abs(F_gpu - F_or) <= 1e-5 * F_or


# Per-worker minibatch losses of the non-IID configuration are ill-conditioned: two
# runs of the ORACLE that differ only in bf16 operand rounding already disagree by
# up to 0.39 on a single worker's loss (10 %) and by 3.3 % on the parameters after
# 24 iterations, while their mean over the 64 workers agrees to 0.3 %.  So config 4
# is compared on the worker-mean loss; config 3 also element by element.
@pytest.mark.parametrize("name,iters,tol_param,per_worker", [("c3", 12, 2e-2, True),
                                                             ("c4", 16, 8e-2, False)])
def test_mlp_configs_first_iterations_against_exact_oracle(name, iters, tol_param, per_worker):
    table = None
    if name == "c4":
        from paper_2002_09539_b200 import class_pairs
        table = class_pairs(0, si.CONFIGS[name]["m"], device="cpu").numpy()
        assert np.array_equal(table, sampling.class_pairs(0, si.CONFIGS[name]["m"]))
    c, X, y, x0, opt, lg = _gpu(name, iters, table)
    st, lo, _ = _oracle(c, X, y, x0, iters)       # exact fp64, no operand rounding
    assert np.isfinite(lg).all()
    mean_g, mean_o = lg.mean(axis=1), lo.mean(axis=1)
    assert np.abs(mean_g - mean_o).max() <= TOL_BF16_LOSS * np.abs(mean_o).max()
    assert (np.abs(mean_g - mean_o) <= TOL_BF16_LOSS * mean_o).all()
    if per_worker:
        assert np.abs(lg - lo).max() <= TOL_BF16_LOSS * np.abs(lo).max()
    assert state_err(opt, st) <= tol_param
    xbar = opt.get_params(-4)
    idx = np.random.default_rng(0).integers(0, X.shape[1], size=(c["m"], 256))
    Xs = np.stack([X[i][idx[i]] for i in range(c["m"])])
    ys = np.stack([y[i][idx[i]] for i in range(c["m"])])
    F_gpu = models.full_objective("mlp", c["dims"], xbar, Xs, ys)
    F_or = models.full_objective("mlp", c["dims"], st.mean_model(), Xs, ys)
    assert abs(F_gpu - F_or) <= TOL_BF16_LOSS * F_or


# How long the stored trajectory can be followed.  The momentum configurations are
# chaotic once the loss is small: the SAME kernels started from x0 with 1e-7 added to
# one entry end config 3 with a 40 % different objective, and two fp64 ORACLE runs
# that differ by that perturbation agree to 6 digits up to iteration 250, by 1 % at 400,
# 3 % at 450, 45 % at 700 and end 22 % apart (tests/golden/c3_final.json vs
# c3_perturbed.json).  The bf16 path gets there sooner, because a last-bit difference in
# fp32 can flip an operand by a whole bf16 ulp: five GPU runs whose x0 differs by 1e-7 in
# one entry agree on the 50-iteration block means of config 3 to 0.15 % up to iteration 150
# and spread by 2 % over iterations 151-200 and by 4 % over 201-250.
# No implementation can meet a 2e-2 bound on the loss after the full 1000 iterations,
# so the bound is enforced on the stored checkpoints up to STRICT_UNTIL and the end of
# the run is checked for having trained to the same level.
# Config 4 (tau = 8, alpha = 0.5) stays reproducible to the end, so there the 2e-2 bound is
# enforced on every checkpoint and on the final objective.
STRICT_UNTIL = {"c3": 150, "c4": 800}          # one iteration's worker-mean loss
STRICT_BLOCKS_UNTIL = {"c3": 150, "c4": 800}   # mean over blocks of 50 iterations
FINAL_STRICT = {"c3": False, "c4": True}


@pytest.mark.parametrize("name", ["c3", "c4"])
def test_mlp_configs_full_length(name):
    path = os.path.join(GOLDEN, name + "_final.json")
    if not os.path.exists(path):
        pytest.skip("stored oracle result %s has not been generated yet" % path)
    gold = json.load(open(path))
    table = sampling.class_pairs(0, si.CONFIGS[name]["m"]) if name == "c4" else None
    c, X, y, x0, opt, lg = _gpu(name, gold["iters"], table)
    assert np.isfinite(lg).all()
    every50 = lg.mean(axis=1)[49::50]
    for t, want in enumerate(gold["minibatch_loss_mean_every_50"]):
        k = 50 * (t + 1)
        if k <= STRICT_UNTIL[name]:
            assert abs(every50[t] - want) <= TOL_BF16_LOSS * want, (k, every50[t], want)
    blocks = gold.get("minibatch_loss_block_mean_50", [])
    for t, want in enumerate(blocks):
        if 50 * (t + 1) <= STRICT_BLOCKS_UNTIL[name]:
            got = float(lg[50 * t:50 * t + 50].mean())
            assert abs(got - want) <= TOL_BF16_LOSS * want, (50 * (t + 1), got, want)
    xbar, z = opt.get_params(-4).copy(), opt.get_params(-1).copy()
    F_mean = models.full_objective("mlp", c["dims"], xbar, X, y)
    F_anchor = models.full_objective("mlp", c["dims"], z, X, y)
    if FINAL_STRICT[name]:
        assert abs(F_mean - gold["F_mean_model"]) <= TOL_BF16_LOSS * gold["F_mean_model"], F_mean
        assert abs(F_anchor - gold["F_anchor"]) <= TOL_BF16_LOSS * gold["F_anchor"], F_anchor
    else:
        # the chaotic end of the run: six GPU runs that differ by 1e-7 in one entry of x0 end
        # with F(mean model) between 0.11 and 0.35 and F(anchor) between 0.12 and 1.15 (the
        # anchor carries momentum 0.9), the tail of the training loss between 0.14 and 0.20
        # and the parameter norm within 0.3 %.  Only the stable statistics are held tightly.
        assert 0.25 * gold["F_mean_model"] <= F_mean <= 4.0 * gold["F_mean_model"], F_mean
        assert np.isfinite(F_anchor) and F_anchor < float(lg[0].mean())
        tail = float(lg[-50:].mean())
        assert 0.5 * gold["minibatch_loss_last10_mean"] <= tail <= 2.0 * gold["minibatch_loss_last10_mean"]
    # it trained: the minibatch loss at the end is far below the first iteration's
    assert float(lg[-10:].mean()) < 0.5 * float(lg[0].mean())
    assert abs(np.linalg.norm(xbar) - gold["norm2_mean_model"]) <= 0.02 * gold["norm2_mean_model"]


@pytest.mark.parametrize("name,gemm", [("c3", 1), ("c4", 1), ("c3", 3)])
def test_anchor_fusion_at_full_size_gives_the_bits_of_the_worker_mean_kernel(name, gemm):
    # configs 3 and 4 as bench.py runs them (replayed graph blocks), with the worker sum inside
    # the sync-step weight-gradient launch (gemm_bf16 = 1) or inside the stand-alone update
    # kernel (gemm_bf16 = 3), and with the worker-mean kernel: identical bits
    from paper_2002_09539_b200 import OverlapLocalSGD
    c = si.CONFIGS[name]
    P = sum(o * i + o for i, o in zip(c["dims"][:-1], c["dims"][1:]))
    weights = sum(o * i for i, o in zip(c["dims"][:-2], c["dims"][1:-1]))   # hidden layers
    table = sampling.class_pairs(0, c["m"]) if name == "c4" else None
    X, y = si.mixture_data(0, c["m"], c["n"], c["dims"][0], table)
    x0 = si.model_init(0, "mlp", c["dims"])
    Xd, yd = to_dev(X), to_dev(y)
    iters = 5 * c["tau"] * (4 if c["tau"] == 2 else 1)
    got = {}
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    for fused in (True, False):
        with torch.cuda.stream(stream):
            opt = OverlapLocalSGD("mlp", m=c["m"], tau=c["tau"], gamma=c["gamma"], alpha=c["alpha"],
                                  beta=c["beta"], mu=c["mu"], batch=c["batch"], seed=0, dims=c["dims"],
                                  gemm_bf16=gemm, x0=x0, X=Xd, y=yd)
            opt.set_anchor_fusion(fused)
            loss = torch.zeros((iters, c["m"]), device="cuda")
            opt.run(iters, loss)
            assert opt.graph_replays >= 1
            opt.join()
            assert opt.summed_floats == ((weights if gemm == 1 else P) if fused else 0)
        torch.cuda.synchronize()
        z, v = opt.get_params(-1).copy(), opt.get_params(-2).copy()
        xs = [opt.get_params(i).copy() for i in (0, c["m"] // 2, c["m"] - 1)]
        got[fused] = [z, v, loss.cpu().numpy()] + xs
        opt.close()
    for a, b in zip(got[True], got[False]):
        assert np.array_equal(a, b)


def test_config3_late_regime_resynchronised_with_the_oracle():
    """Config 3 beyond the point where its trajectory stops being reproducible: the small-loss,
    large-momentum regime of iterations 300-1000.  Chaos cannot be followed over hundreds of
    iterations, but ten can: at the period boundaries k0 the device's whole state (x_i, u_i, z,
    v) is read back and handed to a fresh oracle as ITS start, exactly as x0 is at k = 0 (an
    input to both sides, no expected value comes from the device); both then run ten
    iterations on the rule's own minibatches.

    Held to the 2e-2 bar of the bf16 paths: against the EXACT fp64 oracle, every iteration's
    worker-mean loss (relative) and every per-worker loss (on the scale of the window's
    largest loss, the yardstick of the first-iterations test above); against the oracle with
    the configuration's own operand rounding, every single per-worker loss relative to
    itself.  The last is not asked of the exact oracle because the two ORACLES already differ
    by up to 2.2 % on single entries there (measured: 1.1 %, 1.0 %, 2.2 % at k0 = 300, 600,
    900, against 0.6 %, 0.9 %, 1.1 % between the device and the rounded oracle): that is the
    operand rounding acting on one worker's small minibatch loss, not the kernels."""
    import copy
    from paper_2002_09539_b200 import OverlapLocalSGD
    c = si.CONFIGS["c3"]
    m, steps = c["m"], 10
    X, y = si.mixture_data(0, m, c["n"], c["dims"][0])
    x0 = si.model_init(0, "mlp", c["dims"])
    opt = OverlapLocalSGD("mlp", m=m, tau=c["tau"], gamma=c["gamma"], alpha=c["alpha"],
                          beta=c["beta"], mu=c["mu"], batch=c["batch"], seed=0, dims=c["dims"],
                          gemm_bf16=c["gemm_bf16"], x0=x0, X=to_dev(X), y=to_dev(y))
    kw = dict(m=m, tau=c["tau"], batch=c["batch"], gamma=c["gamma"], alpha=c["alpha"],
              beta=c["beta"], mu=c["mu"], seed=0, iters=steps)
    first_loss = None
    for k0 in (300, 600, 900):
        warm = torch.zeros((k0 - opt.iteration, m), device="cuda")
        opt.run(k0 - opt.iteration, warm)        # long run: replayed graph blocks, as bench.py
        if first_loss is None:
            first_loss = float(warm[0].mean())
        assert opt.iteration == k0
        st = olsgd.OverlapLocalSGD(x0, m, c["tau"], c["gamma"], c["alpha"], c["beta"], c["mu"])
        st.x = np.stack([opt.get_params(i).copy() for i in range(m)]).astype(np.float64)
        st.u = np.stack([opt.get_params(-5 - i).copy() for i in range(m)]).astype(np.float64)
        st.z = opt.get_params(-1).astype(np.float64)
        st.v = opt.get_params(-2).astype(np.float64)
        st.k = k0
        st_rounded = copy.deepcopy(st)
        x_start, z_start = st.x.copy(), st.z.copy()
        # the regime the test is about: trained far below the start, momentum buffers loaded
        assert float(warm[-10:].mean()) < 0.5 * first_loss
        assert np.abs(st.u).max() > 0 and np.abs(st.v).max() > 0
        lg = torch.zeros((steps, m), device="cuda")
        opt.run(steps, lg)
        lg = lg.cpu().numpy()
        st, lo, _ = runner.run_model("mlp", c["dims"], X, y, None, state=st, **kw)
        st_rounded, lr, _ = runner.run_model("mlp", c["dims"], X, y, None, state=st_rounded,
                                             bf16_operands=True, **kw)
        assert st.k == opt.iteration == k0 + steps
        # exact oracle: worker-mean loss of every iteration, relative
        mean_g, mean_o = lg.mean(axis=1), lo.mean(axis=1)
        assert (np.abs(mean_g - mean_o) <= TOL_BF16_LOSS * mean_o).all(), (k0, mean_g, mean_o)
        # exact oracle: every per-worker loss on the scale of the window, and none far off
        assert np.abs(lg - lo).max() <= TOL_BF16_LOSS * np.abs(lo).max(), (k0, np.abs(lg - lo).max())
        assert (np.abs(lg - lo) <= 5e-2 * lo).all(), (k0, (np.abs(lg - lo) / lo).max())
        # oracle with the operand rounding of the configuration: every per-worker loss, relative
        assert (np.abs(lg - lr) <= TOL_BF16_LOSS * lr).all(), (k0, (np.abs(lg - lr) / lr).max())
        assert state_err(opt, st) <= TOL_BF16_LOSS, (k0, state_err(opt, st))
        assert state_err(opt, st_rounded) <= TOL_BF16_LOSS, (k0, state_err(opt, st_rounded))
        # the ten steps themselves (not the state they started from) agree as well
        xg, zg, _ = opt.state()
        moved_o = np.abs(st.x - x_start).max()
        assert np.abs((xg - x_start) - (st.x - x_start)).max() <= 0.1 * moved_o, k0
        assert np.abs((zg - z_start) - (st.z - z_start)).max() <= 0.1 * np.abs(st.z - z_start).max(), k0
    opt.close()


@pytest.mark.parametrize("m", [8, 16, 64])
def test_config5_parity_size_point(m):
    from paper_2002_09539_b200 import OverlapLocalSGD
    c = si.CONFIGS["c5"]
    P, iters = 1_000_000, 2 * c["tau"] + 1
    x0 = si.flat_init(0, P)
    grads = [si.flat_grads(0, k, m, P, c["grad_std"]) for k in range(iters)]
    st = runner.run_flat(x0, grads, m=m, tau=c["tau"], gamma=c["gamma"], alpha=c["alpha"],
                         beta=c["beta"], mu=c["mu"])
    opt = OverlapLocalSGD("flat", m=m, tau=c["tau"], gamma=c["gamma"], alpha=c["alpha"],
                          beta=c["beta"], mu=c["mu"], flat_P=P, x0=x0)
    for k in range(iters):
        opt.local_step_with_grads(to_dev(grads[k]))
        if (k + 1) % c["tau"] == 0:
            opt.period_sync()
    assert state_err(opt, st) <= 1e-5


def test_config5_largest_point_on_sampled_columns():
    # P = 50M, m = 64 as bench.py runs it.  The update is separable per parameter,
    # so the oracle runs exactly on a random sample of columns.
    from paper_2002_09539_b200 import OverlapLocalSGD
    c = si.CONFIGS["c5"]
    P, m, iters = 50_000_000, 64, 2 * c["tau"] + 1
    gen = torch.Generator(device="cuda").manual_seed(1)
    x0 = torch.randn(P, device="cuda", generator=gen)
    cols = torch.from_numpy(np.sort(np.random.default_rng(2).choice(P, 4096, replace=False))).cuda()
    cols[0], cols[-1] = 0, P - 1
    opt = OverlapLocalSGD("flat", m=m, tau=c["tau"], gamma=c["gamma"], alpha=c["alpha"],
                          beta=c["beta"], mu=c["mu"], flat_P=P, x0=x0)
    st = olsgd.OverlapLocalSGD(x0[cols].cpu().numpy(), m, c["tau"], c["gamma"], c["alpha"],
                               c["beta"], c["mu"])
    g = torch.empty((m, P), device="cuda")
    for k in range(iters):
        g.normal_(0.0, c["grad_std"], generator=gen)
        st.step(g[:, cols].cpu().numpy())
        opt.local_step_with_grads(g)
        if (k + 1) % c["tau"] == 0:
            opt.period_sync()
    out = torch.empty(P, device="cuda")
    got = []
    for which in list(range(0, m, 9)) + [m - 1, -1]:
        opt.get_params(which, out)
        got.append(out[cols].cpu().numpy())
    want = [st.x[i] for i in list(range(0, m, 9)) + [m - 1]] + [st.z]
    assert max_rel_err(got, want) <= 1e-5
    opt.get_params(-2, out)
    v = out[cols].cpu().numpy()
    assert np.abs(v - st.v).max() <= 1e-5 * np.abs(st.z).max()
