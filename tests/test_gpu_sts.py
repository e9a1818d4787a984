"""GPU Sequential Temperature Scaling vs the oracle (Section 3.2.1, post-hoc calibration).

The GPU forms the cumulative products and sigmoids in fp32, the oracle in fp64, so a sample within
rounding of a bin edge may fall into the neighbouring bin: an ECE may differ by a few multiples of 1/N.
The chosen temperature must be the oracle's unless the oracle itself rates the two candidates within that
same tolerance of each other.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _gpu(conf, acc, ver, grid, n_bins):
    N, gamma = conf.shape
    G = grid.numel()
    T = torch.full((gamma,), -1.0, device="cuda")
    eb = torch.full((gamma,), -1.0, dtype=torch.float64, device="cuda")
    ea = torch.full((gamma,), -1.0, dtype=torch.float64, device="cuda")
    eg = torch.full((gamma, G), -1.0, dtype=torch.float64, device="cuda")
    ws = B.workspace(B.dspark_sts_workspace_bytes(N, gamma, G, n_bins)).fill_(0xFF)
    B.dspark_sts_calibrate(conf, acc, grid, n_bins, verified_len=ver, out_T=T, out_ece_before=eb, out_ece_after=ea,
                           out_ece_grid=eg, workspace=ws)
    torch.cuda.synchronize()
    return T.cpu().numpy(), eb.cpu().numpy(), ea.cpu().numpy(), eg.cpu().numpy()


@pytest.mark.parametrize("N,gamma,G,n_bins,partial", [(20_000, 8, 33, 15, True), (3_001, 5, 7, 10, False),
                                                     (150_000, 16, 65, 15, True), (64, 3, 4, 2, True)])
def test_against_oracle(N, gamma, G, n_bins, partial):
    conf, acc, ver = W.sts_input(N, gamma, 40 + gamma, "cuda", partial=partial)
    grid = torch.tensor(np.geomspace(0.4, 5.0, G), dtype=torch.float32, device="cuda")
    T, eb, ea, eg = _gpu(conf, acc, ver if partial else None, grid, n_bins)
    oT, oeb, oea, oeg = oracle.sts_calibrate(conf.cpu().numpy(), acc.cpu().numpy(), grid.cpu().numpy(), n_bins,
                                             verified_len=ver.cpu().numpy() if partial else None)
    tol = 1e-6 + 8.0 / N
    gnp = grid.cpu().numpy()
    for k in range(gamma):
        assert abs(eb[k] - oeb[k]) <= tol
        if T[k] != oT[k]:
            # allowed only if the oracle rates the GPU's choice as good as its own within the tolerance; the
            # chains differ from here on, so the later positions are not comparable
            g_gpu = int(np.argmin(np.abs(gnp - T[k])))
            assert oeg[k, g_gpu] - oeg[k].min() <= 2 * tol, (k, T[k], oT[k])
            break
        np.testing.assert_allclose(eg[k], oeg[k], atol=tol)
        assert abs(ea[k] - oea[k]) <= tol
    else:
        np.testing.assert_array_equal(T, oT)
    print(f"[sts] N={N} gamma={gamma}: T = {np.round(T, 3).tolist()}, ECE {eb.max():.4f} -> {ea.max():.4f}")


def test_recovers_the_overconfidence_factor_and_apply():
    N, gamma = 200_000, 6
    conf, acc, ver = W.sts_input(N, gamma, 7, "cuda", overconfidence=2.0, partial=False)
    grid = torch.tensor(np.geomspace(0.5, 4.0, 49), dtype=torch.float32, device="cuda")
    T, eb, ea, _ = _gpu(conf, acc, None, grid, 15)
    assert np.all(np.abs(T - 2.0) <= 0.25), T
    assert np.all(ea < 0.3 * eb) and np.all(ea < 0.01)
    out = torch.empty_like(conf)
    B.dspark_sts_apply(conf, torch.tensor(T, device="cuda"), out)
    torch.cuda.synchronize()
    want = oracle.sts_apply(conf.cpu().numpy(), T)
    assert np.abs(out.cpu().numpy().astype(np.float64) - want).max() <= 2e-6
    # order inside a position is kept
    c0, o0 = conf[:5000, 0].cpu().numpy(), out[:5000, 0].cpu().numpy()
    assert np.all(np.diff(o0[np.argsort(c0, kind="stable")]) >= 0)


def test_edge_values_and_unverified_positions():
    conf = torch.tensor([[0.0, 0.5, 0.9], [1.0, 0.25, 0.9], [float("nan"), 0.75, 0.9], [1.5, 0.5, 0.9]], device="cuda")
    acc = torch.tensor([0, 2, 0, 1], dtype=torch.int32, device="cuda")
    ver = torch.tensor([2, 2, 1, 2], dtype=torch.int32, device="cuda")
    grid = torch.tensor([0.5, 1.0, 2.0], device="cuda")
    T, eb, ea, eg = _gpu(conf, acc, ver, grid, 4)
    oT, oeb, oea, oeg = oracle.sts_calibrate(conf.cpu().numpy(), acc.cpu().numpy(), grid.cpu().numpy(), 4,
                                             verified_len=ver.cpu().numpy())
    np.testing.assert_array_equal(T, oT)
    np.testing.assert_allclose(eb, oeb, atol=1e-6)
    np.testing.assert_allclose(eg, oeg, atol=1e-6)
    assert T[2] == 1.0 and ea[2] == 0.0          # nobody verified position 2
    out = torch.empty_like(conf)
    B.dspark_sts_apply(conf, torch.tensor([3.0, 1.0, 2.0], device="cuda"), out)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(out[:, 0].cpu().numpy(), [0.0, 1.0, 0.0, 1.0])
    np.testing.assert_allclose(out[:, 1].cpu().numpy(), [0.5, 0.25, 0.75, 0.5], rtol=1e-6)


def test_unusable_grid_temperatures_are_never_chosen():
    # a grid with a zero, a negative, a NaN and an infinite entry among good ones: the good entries are rated as
    # without the bad ones, the bad ones are marked NaN and never win
    rng = np.random.default_rng(3)
    N, gamma = 5000, 4
    conf = torch.from_numpy(rng.uniform(0.05, 0.95, size=(N, gamma)).astype(np.float32)).cuda()
    acc = torch.from_numpy(rng.integers(0, gamma + 1, size=N).astype(np.int32)).cuda()
    good = [0.5, 0.8, 1.0, 1.5, 2.5]
    mixed = torch.tensor([0.0, 0.5, -1.0, 0.8, float("nan"), 1.0, float("inf"), 1.5, 2.5], device="cuda")
    Tg, _, eag, egg = _gpu(conf, acc, None, torch.tensor(good, device="cuda"), 10)
    Tm, _, eam, egm = _gpu(conf, acc, None, mixed, 10)
    np.testing.assert_array_equal(Tm, Tg)
    np.testing.assert_allclose(eam, eag, atol=1e-12)
    assert np.isnan(egm[:, [0, 2, 4, 6]]).all()
    np.testing.assert_allclose(egm[:, [1, 3, 5, 7, 8]], egg, atol=1e-12)
    bad_only = torch.tensor([0.0, float("nan")], device="cuda")
    Tb, _, _, _ = _gpu(conf, acc, None, bad_only, 10)
    np.testing.assert_array_equal(Tb, np.ones(gamma, dtype=np.float32))
