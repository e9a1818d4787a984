"""GPU scheduler vs the CPU oracle: bit-exact lengths, survival products, offsets, info."""
import numpy as np
import pytest
import torch

import helpers as H
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu
MODES = [B.DSPARK_SCHED_EARLY_STOP, B.DSPARK_SCHED_GLOBAL, B.DSPARK_SCHED_TOPK]


@pytest.mark.parametrize("mode", MODES)
def test_config_1(mode):
    sched, _ = W.config_1("cuda")
    g, o = H.check_schedule(sched, mode, topk=5)
    assert g["info"].B <= 16


@pytest.mark.parametrize("mode", MODES)
def test_config_3_full_size(mode):
    g, o = H.check_schedule(W.config_3_schedule("cuda"), mode, topk=300)
    assert g["info"].B <= 1024 and g["lengths"].max() <= 16


@pytest.mark.parametrize("mode", MODES)
def test_config_5_full_size(mode):
    g, o = H.check_schedule(W.config_5_schedule("cuda"), mode, topk=2000)
    assert g["info"].B <= 4096
    if mode == B.DSPARK_SCHED_GLOBAL:
        e, _ = H.check_schedule(W.config_5_schedule("cuda"), B.DSPARK_SCHED_EARLY_STOP)
        assert e["info"].n_admitted < g["info"].n_admitted      # profile P5 has a kink: early != global


def test_appendix_a_on_gpu(golden):
    g = golden("appendix_a.txt")
    sps = [float(x) for x in g["sps"]]
    for case in ("case1", "case2"):
        conf = torch.tensor([[float(g["a1"][0]), float(g[f"{case}_c2"][0])]], dtype=torch.float32)
        s = W.ScheduleInput(conf, [1, 2, 3], sps, budget_tokens=3, max_tokens=3)
        e, _ = H.check_schedule(s, B.DSPARK_SCHED_EARLY_STOP)
        gl, _ = H.check_schedule(s, B.DSPARK_SCHED_GLOBAL)
        assert int(e["lengths"][0]) == int(g[f"{case}_len_early"][0])
        assert int(gl["lengths"][0]) == int(g[f"{case}_len_global"][0])


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes_ties_and_jagged_profiles(seed):
    rng = np.random.default_rng(seed)
    R = int(rng.integers(1, 700))
    gamma = int(rng.integers(1, 24))
    conf = rng.uniform(0.05, 1.0, size=(R, gamma)).astype(np.float32)
    conf[rng.random((R, gamma)) < 0.1] = 1.0                       # ties
    conf[rng.random((R, gamma)) < 0.02] = 0.0                      # blocks that end early
    if R > 3:
        conf[1] = conf[2]
    n_bp = 12
    toks = np.sort(rng.choice(np.arange(1, R * (gamma + 1) + 2), size=n_bp, replace=False)).tolist()
    sps = rng.uniform(5, 100, n_bp)
    if seed % 2 == 0:
        sps = np.sort(sps)[::-1]
    budget = int(rng.integers(R, R * (gamma + 1) + 1))
    s = W.ScheduleInput(torch.from_numpy(conf), toks, sps.tolist(), budget, max_tokens=R * (gamma + 1))
    for mode in MODES:
        H.check_schedule(s, mode, topk=int(rng.integers(0, R * gamma + 1)))
    dl = rng.integers(0, gamma + 1, size=R).astype(np.int32)
    H.check_schedule(s, B.DSPARK_SCHED_GLOBAL, draft_len=dl)


def test_edge_cases():
    # bad confidences are clamped with a warning bit; budget below R yields all zeros
    conf = torch.tensor([[0.9, float("nan"), 0.9], [1.5, -0.1, 0.3], [0.5, 0.5, 0.5]], dtype=torch.float32)
    s = W.ScheduleInput(conf, [1, 12], [10.0, 9.0], budget_tokens=12, max_tokens=12)
    g, _ = H.check_schedule(s, B.DSPARK_SCHED_EARLY_STOP)
    assert g["info"].status & B.DEV_CONF_CLAMPED
    s.budget_tokens = 2
    g, _ = H.check_schedule(s, B.DSPARK_SCHED_GLOBAL)
    assert (g["lengths"] == 0).all() and g["info"].status & B.DEV_BUDGET_LT_R
    # one request, one position; large key count beyond shared memory (global-memory keys)
    H.check_schedule(W.ScheduleInput(torch.tensor([[0.7]]), [1, 2], [3.0, 2.9], 2, 2), B.DSPARK_SCHED_EARLY_STOP)
    rng = np.random.default_rng(0)
    big = torch.from_numpy(rng.uniform(0.3, 1.0, size=(2048, 12)).astype(np.float32))    # 24576 keys > 16384
    H.check_schedule(W.ScheduleInput(big, [1, 30000], [100.0, 20.0], 9000, 30000), B.DSPARK_SCHED_GLOBAL)
    # lookups beyond max_tokens use the last table entry
    H.check_schedule(W.ScheduleInput(big[:64], [1, 100], [50.0, 40.0], 10**6, 100), B.DSPARK_SCHED_GLOBAL)


def test_selection_path_with_mass_ties():
    # large candidate set + small cap: the library ranks only the candidates that fit under the cap;
    # here thousands of candidates share the same survival value, so the cap falls inside a tie group
    rng = np.random.default_rng(11)
    R, gamma = 640, 16                                     # 10 240 entries
    conf = rng.choice([1.0, 0.5, 0.75], size=(R, gamma), p=[0.5, 0.3, 0.2]).astype(np.float32)
    conf[:, 0] = 1.0
    for budget in (R + 100, R + 1777, R + 5000):
        s = W.ScheduleInput(torch.from_numpy(conf), [1, 20000], [100.0, 40.0], budget, max_tokens=20000)
        for mode in MODES:
            H.check_schedule(s, mode, topk=1500)
    # continuous values, cap well below half of the candidates
    conf = rng.uniform(0.2, 1.0, size=(1024, 16)).astype(np.float32)
    s = W.ScheduleInput(torch.from_numpy(conf), [1, 4000, 20000], [90.0, 60.0, 10.0], 1024 + 3000, max_tokens=20000)
    for mode in MODES:
        H.check_schedule(s, mode, topk=2999)


@pytest.mark.parametrize("R,gamma", [(37, 40), (300, 64), (130, 100), (9, 33)])
def test_blocks_longer_than_a_tile(R, gamma):
    # gamma > 32: a request spans several 32-entry tiles
    rng = np.random.default_rng(R * gamma)
    conf = rng.uniform(0.55, 1.0, size=(R, gamma)).astype(np.float32)
    conf[rng.random((R, gamma)) < 0.05] = 1.0
    conf[rng.random((R, gamma)) < 0.01] = 0.0
    toks = [1, R, 2 * R, 4 * R, R * (gamma + 1)]
    s = W.ScheduleInput(torch.from_numpy(conf), toks, [100.0, 90.0, 70.0, 45.0, 5.0],
                        budget_tokens=R * (gamma // 2), max_tokens=R * (gamma + 1))
    for mode in MODES:
        H.check_schedule(s, mode, topk=R * 7)
    dl = rng.integers(0, gamma + 1, size=R).astype(np.int32)
    H.check_schedule(s, B.DSPARK_SCHED_EARLY_STOP, draft_len=dl)


def test_host_side_errors():
    prof = B.Profile([1, 8], [2.0, 1.0], 8)
    conf = torch.rand(4, 4, device="cuda")
    out = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(B.DsparkError, match="workspace"):
        B.dspark_schedule(prof, conf, 8, out_len=out, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    ws = B.workspace(B.dspark_schedule_workspace_bytes(4, 4))
    with pytest.raises(B.DsparkError, match="invalid"):
        B.dspark_schedule(prof, conf, 8, mode=9, out_len=out, workspace=ws)
    with pytest.raises(B.DsparkError):
        B.Profile([4, 4], [1.0, 2.0], 8)
    prof.close()


def test_build_offsets():
    lengths = torch.randint(0, 9, (1500,), dtype=torch.int32, device="cuda")
    off = torch.zeros(1501, dtype=torch.int32, device="cuda")
    B.dspark_build_offsets(lengths, off)
    want = torch.cat([torch.zeros(1, dtype=torch.int64, device="cuda"), torch.cumsum(lengths.long() + 1, 0)])
    assert torch.equal(off.long(), want)
