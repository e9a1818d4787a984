"""Asynchronous top-K scheduling (Section 5.2) on the GPU: device-resident state across steps,
bit-exact against the oracle, and the schedule -> verify chain replayed from a CUDA graph."""
import numpy as np
import pytest
import torch

import helpers as H
import oracle
from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _conf(step, R, gamma, device="cuda"):
    g = torch.Generator(device=device); g.manual_seed(900 + step)
    i = torch.arange(1, gamma + 1, device=device, dtype=torch.float32)
    shift = 2.0 - 0.25 * i + 0.4 * np.sin(step)                    # the load drifts from step to step
    return torch.sigmoid(torch.randn(R, gamma, generator=g, device=device) + shift).float().contiguous()


@pytest.mark.parametrize("R,gamma,budget,K0", [(256, 16, 1024, 300), (512, 32, 4096, 1000), (5, 3, 12, 2)])
def test_state_lives_on_the_device_across_steps(R, gamma, budget, K0):
    bp = W.PROFILE_P5 if budget == 4096 else ([1, max(2, budget // 2), budget], [100.0, 80.0, 30.0])
    prof = B.Profile(bp[0], bp[1], budget)
    table = oracle.sps_table(bp[0], bp[1], budget)
    state = torch.full((4,), -1, dtype=torch.int32, device="cuda")
    B.dspark_async_state_init(state, K0)
    host_state = np.array([0, K0, K0], dtype=np.int32)
    out_len = torch.zeros(R, dtype=torch.int32, device="cuda")
    off = torch.zeros(R + 1, dtype=torch.int32, device="cuda")
    info = torch.zeros(32, dtype=torch.uint8, device="cuda")
    ws = B.workspace(B.dspark_schedule_workspace_bytes(R, gamma)).fill_(0xFF)
    ks = []
    for step in range(7):
        conf = _conf(step, R, gamma)
        B.dspark_schedule_async(prof, conf, budget, state, out_len=out_len, out_row_offsets=off, out_info=info,
                                workspace=ws)
        o = oracle.schedule_async(conf.cpu().numpy(), table, budget, host_state)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(out_len.cpu().numpy(), o.lengths)
        np.testing.assert_array_equal(off.cpu().numpy(), np.concatenate([[0], np.cumsum(o.lengths + 1)]))
        i = B.read_sched_info(info)
        assert (i.B, i.n_admitted, i.n_candidates) == (o.B, o.n_admitted, o.n_candidates)
        assert i.tau == o.tau and i.theta == o.theta
        np.testing.assert_array_equal(state.cpu().numpy()[:3], host_state)
        ks.append(o.n_admitted)
        # the capacity in force is the global optimum of two steps ago
        if step >= 2:
            g = oracle.schedule(_conf(step - 2, R, gamma).cpu().numpy(), table, budget, oracle.MODE_GLOBAL)
            assert o.n_admitted == min(g.n_admitted, o.n_candidates, budget - R)
    assert len(set(ks[2:])) > 1 or R < 10           # the capacity really follows the drifting load
    prof.close()


def test_schedule_then_verify_replayed_from_a_cuda_graph():
    R, gamma, V, budget, K0 = 32, 8, 8192, 160, 60
    bp = ([1, 80, 160], [100.0, 85.0, 40.0])
    prof = B.Profile(bp[0], bp[1], budget)
    table = oracle.sps_table(bp[0], bp[1], budget)
    cap_rows = budget                                         # B = R + sum l_r <= budget rows
    # static buffers the graph reads and writes
    conf_buf = torch.zeros(R, gamma, device="cuda")
    target_buf = torch.zeros(cap_rows, V, dtype=torch.bfloat16, device="cuda")
    draft_buf = torch.zeros(cap_rows, V, dtype=torch.bfloat16, device="cuda")
    tok_buf = torch.zeros(cap_rows, dtype=torch.int32, device="cuda")
    state = torch.zeros(4, dtype=torch.int32, device="cuda")
    out_len = torch.zeros(R, dtype=torch.int32, device="cuda")
    off = torch.zeros(R + 1, dtype=torch.int32, device="cuda")
    acc = torch.zeros(R, dtype=torch.int32, device="cuda")
    out = torch.zeros(cap_rows, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sws = B.workspace(B.dspark_schedule_workspace_bytes(R, gamma))
    vws = B.workspace(B.dspark_verify_workspace_bytes(R, cap_rows, V))

    def chain():
        B.dspark_schedule_async(prof, conf_buf, budget, state, out_len=out_len, out_row_offsets=off, workspace=sws)
        B.dspark_verify(target_buf, draft_buf, off, tok_buf, 0.9, 77, accepted_len=acc, out_tokens=out,
                        dev_status=status, workspace=vws, n_rows=cap_rows)

    # one eager pass (also sets kernel attributes), then capture; the capture itself executes nothing
    conf_buf.copy_(_conf(100, R, gamma))
    off.copy_(torch.arange(R + 1, dtype=torch.int32))
    B.dspark_async_state_init(state, K0)
    chain()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        chain()
    B.dspark_async_state_init(state, K0)
    host_state = np.array([0, K0, K0], dtype=np.int32)
    torch.cuda.synchronize()

    for step in range(5):
        conf = _conf(step, R, gamma)
        o = oracle.schedule_async(conf.cpu().numpy(), table, budget, host_state)
        batch = W.sampling_batch(torch.from_numpy(o.lengths), V, 3000 + step, "cuda", temperature=0.9, verify_seed=77)
        conf_buf.copy_(conf)
        target_buf[: batch.n_rows].copy_(batch.target)
        draft_buf[: batch.draft.shape[0]].copy_(batch.draft)
        tok_buf[: batch.n_rows].copy_(batch.draft_tokens)
        status.zero_()
        graph.replay()                                        # schedule + verify, no host decision in between
        torch.cuda.synchronize()
        np.testing.assert_array_equal(out_len.cpu().numpy(), o.lengths)
        assert torch.equal(off.cpu(), batch.row_offsets.cpu())
        ov = H.oracle_verify(batch, eval_all=False)
        g = dict(acc=acc.cpu().numpy(), out=out.cpu().numpy(), status=int(status.item()), p=None, q=None)
        mism = H.compare_sampling(g, ov, batch.row_offsets.cpu().numpy(), check_probs=False)
        assert mism == 0
        np.testing.assert_array_equal(state.cpu().numpy()[:3], host_state)
    prof.close()
