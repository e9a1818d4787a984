"""Host-side checks of the seeded input generators (CPU): determinism, shapes, the ragged layout invariants
the verifiers rely on.  The generators hold none of the method's arithmetic; these tests only pin their
contract."""
import numpy as np
import torch

from paper_2607_05147_b200 import workloads as W


def test_sampling_batch_is_deterministic_and_well_formed():
    lengths = torch.tensor([3, 0, 2, 5])
    a = W.sampling_batch(lengths, 777, 13, "cpu", temperature=0.8, block=6)
    b = W.sampling_batch(lengths, 777, 13, "cpu", temperature=0.8, block=6)
    assert torch.equal(a.target.view(torch.int16), b.target.view(torch.int16))
    assert torch.equal(a.draft.view(torch.int16), b.draft.view(torch.int16))
    assert torch.equal(a.draft_tokens, b.draft_tokens)
    off = a.row_offsets.numpy()
    np.testing.assert_array_equal(np.diff(off), lengths.numpy() + 1)
    assert a.n_rows == int(off[-1]) and a.V == 777 and a.R == 4
    assert a.draft_row_start is not None and a.draft.shape[0] >= 4 * 6
    np.testing.assert_array_equal(a.draft_row_start.numpy(), np.arange(4) * 6)
    toks = a.draft_tokens.numpy()
    for r in range(4):
        assert ((toks[off[r]:off[r] + lengths[r]] >= 0) & (toks[off[r]:off[r] + lengths[r]] < 777)).all()
    c = W.sampling_batch(lengths, 777, 14, "cpu", temperature=0.8, block=6)
    assert not torch.equal(a.target.view(torch.int16), c.target.view(torch.int16))


def test_compact_layout_has_one_draft_row_per_draft_position():
    lengths = torch.tensor([2, 2, 0, 1])
    b = W.sampling_batch(lengths, 300, 5, "cpu")
    assert b.draft_row_start is None and b.draft.shape[0] == int(lengths.sum())
    assert b.target.shape[0] == int(lengths.sum()) + 4


def test_greedy_batch_and_configs():
    sched, batch = W.config_1("cpu")
    assert sched.conf.shape == (4, 4) and batch.V == 1024 and batch.R == 4 and batch.draft is None
    assert ((sched.conf >= 0.5) & (sched.conf <= 1.0)).all()
    s3 = W.config_3_schedule("cpu")
    assert s3.conf.shape == (256, 16) and s3.budget_tokens == 1024
    s5 = W.config_5_schedule("cpu")
    assert s5.conf.shape == (512, 32) and s5.budget_tokens == 4096


def test_markov_and_sts_inputs():
    m = W.markov_input(5, 640, 3, "cpu", d=16)
    assert m.U.shape == (5, 640) and m.W1.shape == (640, 256) and m.W2.shape == (256, 640)
    assert m.H.shape == (5, 16) and m.w_conf.shape == (16 + 256,) and m.x_prev.dtype == torch.int32
    assert ((m.x_prev >= 0) & (m.x_prev < 640)).all()
    m2 = W.markov_input(5, 640, 3, "cpu", d=16)
    assert torch.equal(m.U.view(torch.int16), m2.U.view(torch.int16)) and torch.equal(m.x_prev, m2.x_prev)
    conf, acc, ver = W.sts_input(1000, 7, 2, "cpu")
    assert conf.shape == (1000, 7) and ((conf > 0) & (conf < 1)).all()
    assert ((acc >= 0) & (acc <= ver)).all() and ((ver >= 1) & (ver <= 7)).all()
    conf2, acc2, ver2 = W.sts_input(1000, 7, 2, "cpu", partial=False)
    assert (ver2 == 7).all()


def test_bf16_bits_roundtrip():
    t = torch.tensor([[1.0, -2.5, 0.0, float("-inf")]], dtype=torch.bfloat16)
    bits = W.bf16_bits(t)
    assert bits.dtype == np.uint16 and bits.tolist() == [[0x3F80, 0xC020, 0x0000, 0xFF80]]
    f = torch.tensor([[1.5, 2.0]])
    assert W.bf16_bits(f).dtype == np.float32
