"""The seeded input recipes are deterministic and have the stated structure."""
import torch

from paper_2409_18747_b200 import synth


def test_deterministic_and_rounded_first():
    a = synth.make_config(3, B=1)
    b = synth.make_config(3, B=1)
    for key in ("q", "k", "v", "m"):
        assert torch.equal(a[key], b[key])
    assert a["q"].dtype == torch.bfloat16 and a["m"].dtype == torch.float32


def test_config3_zero_key_rows():
    c = synth.make_config(3, B=1)
    zero_rows = (c["k"].float().abs().sum(-1) == 0).sum(-1)
    assert (zero_rows == 51).all()  # floor(0.05 * 1024) per (b,h)


def test_config1_row_scales_vary():
    c = synth.make_config(1)
    n = c["q"].norm(dim=-1)
    assert c["q"].dtype == torch.float32 and (n.max() / n.min()) > 50


def test_onehot_case_is_exact():
    c = synth.make_onehot_case(1, 2, 300, 64, torch.bfloat16, 7)
    assert ((c["q"].float() != 0).sum(-1) == 1).all() and ((c["k"].float() != 0).sum(-1) == 1).all()
    assert torch.equal(c["v"].float(), c["v"].float().round())
