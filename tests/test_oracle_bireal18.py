"""Pins for the oracle's Bi-Real Net 18 forward (Section 2.3): each stage is re-computed from the
oracle's own stage INPUT with fp64 library routines (torch), so a wrong stride, padding, shortcut,
BN or ordering in any one stage shows up there; the two convolution forms give identical logits."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from paper_1908_05858_b200 import synth


def bn64(x, bn, eps):
    g, b, m, v = (torch.from_numpy(np.asarray(t)).double().view(1, -1, 1, 1) for t in bn)
    return g * (x - m) / torch.sqrt(v + eps) + b


@pytest.fixture(scope="module")
def run(oracle_mod):
    p = synth.bireal18_params()
    img = synth.bireal18_images(2)
    logits, taps = oracle_mod.bireal18_forward(p, img, conv_form=1, want_taps=True)
    return p, img, logits, taps


def close(a, b, tol=2e-5):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return np.max(np.abs(a - b)) <= tol * (1.0 + np.max(np.abs(b)))


def test_stem_against_fp64(run):
    p, img, _, taps = run
    x = torch.from_numpy(img).double()
    y = F.conv2d(x, torch.from_numpy(p["stem_w"]).double(), stride=2, padding=3)
    y = bn64(y, p["stem_bn"], p["bn_eps"])
    y = F.max_pool2d(y, 3, stride=2, padding=1)
    assert taps[0].shape == (2, 64, 56, 56)
    assert close(taps[0], y.numpy())


def test_every_block_against_fp64(run):
    p, _, _, taps = run
    d = 0
    for b in range(16):
        x = torch.from_numpy(taps[b]).double()  # the oracle's own input to block b
        C = x.shape[1]
        O = synth.STAGE_C[b // 4]
        down = b % 4 == 0 and b > 0
        stride = 2 if down else 1
        xs = torch.where(x < 0, -1.0, 1.0).double()
        ws = torch.where(torch.from_numpy(p["block_w"][b]) < 0, -1.0, 1.0).double()
        acc = F.conv2d(F.pad(xs, (1, 1, 1, 1), value=-1.0), ws, stride=stride)
        y = bn64(acc, p["block_bn"][b], p["bn_eps"])
        if down:
            sc = F.avg_pool2d(x, 2, stride=2)
            sc = F.conv2d(sc, torch.from_numpy(p["down_w"][d]).double().view(O, C, 1, 1))
            sc = bn64(sc, p["down_bn"][d], p["bn_eps"])
            d += 1
        else:
            sc = x
        want = (y + sc).numpy()
        assert taps[b + 1].shape == want.shape == (2, O, synth.STAGE_HW[b // 4], synth.STAGE_HW[b // 4])
        assert close(taps[b + 1], want), b
    assert d == 3


def test_head_against_fp64(run):
    p, _, logits, taps = run
    x = torch.from_numpy(taps[16]).double()
    g = x.mean(dim=(2, 3))
    want = g @ torch.from_numpy(p["fc_w"]).double().t() + torch.from_numpy(p["fc_b"]).double()
    assert logits.shape == (2, 1000)
    assert close(logits, want.numpy())


def test_both_conv_forms_give_identical_logits(oracle_mod, run):
    p, img, logits, _ = run
    l0 = oracle_mod.bireal18_forward(p, img[:1], conv_form=0)
    assert np.array_equal(l0, logits[:1])  # bitwise, and batch-independent


def test_stem_module_against_fp64(oracle_mod):
    """The STEM module variant (Section 2.3; structure = a reading of the missing figure): its output against the same
    structure built from fp64 library routines, and the blocks after it unchanged (same code path as the 7x7 variant)."""
    p = dict(synth.bireal18_params())
    p["stem_module"] = synth.stem_module_params()
    img = synth.bireal18_images(2)
    logits, taps = oracle_mod.bireal18_forward(p, img, conv_form=1, want_taps=True, stem_module=True)
    sm = p["stem_module"]
    x = torch.from_numpy(img).double()
    w = [torch.from_numpy(t).double() for t in sm["w"]]
    s1 = F.relu(bn64(F.conv2d(x, w[0], stride=2, padding=1), sm["bn"][0], p["bn_eps"]))
    a = F.relu(bn64(F.conv2d(s1, w[1]), sm["bn"][1], p["bn_eps"]))
    a = F.relu(bn64(F.conv2d(a, w[2], stride=2, padding=1), sm["bn"][2], p["bn_eps"]))
    b = F.max_pool2d(s1, 2, stride=2)
    y = bn64(F.conv2d(torch.cat([a, b], dim=1), w[3]), sm["bn"][3], p["bn_eps"])
    assert taps[0].shape == (2, 64, 56, 56)
    assert close(taps[0], y.numpy())
    assert (taps[0] < 0).mean() > 0.2 and (taps[0] > 0).mean() > 0.2  # a signed stream: the binary blocks see both signs
    # the head still follows from the last block
    g = torch.from_numpy(taps[16]).double().mean(dim=(2, 3))
    want = g @ torch.from_numpy(p["fc_w"]).double().t() + torch.from_numpy(p["fc_b"]).double()
    assert close(logits, want.numpy())
    # and it is a different network from the 7x7 one
    assert not np.array_equal(logits, oracle_mod.bireal18_forward(p, img, conv_form=1))
