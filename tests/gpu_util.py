"""Helpers shared by the GPU tests: host <-> device marshalling of models and
bit-level comparison.  No arithmetic of the method lives here."""
import numpy as np

from oracle import randes_oracle as ro
from paper_2505_11204_b200 import randes, workloads as wl


def to_dev(a: np.ndarray, device="cuda"):
    import torch

    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(a).to(device)


def from_dev(t) -> np.ndarray:
    import torch

    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def model_to_dev(model):
    return [to_dev(a) for a in model]


def bits(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    return a.view(np.uint32) if a.dtype == np.float32 else a.view(np.uint16)


def assert_bits_equal(got: np.ndarray, want: np.ndarray, what=""):
    g, w = bits(got).ravel(), bits(want).ravel()
    assert g.shape == w.shape, (what, g.shape, w.shape)
    if not np.array_equal(g, w):
        bad = np.flatnonzero(g != w)
        i = int(bad[0])
        raise AssertionError("%s: %d of %d elements differ; first at %d: got %r want %r"
                             % (what, bad.size, g.size, i, got.ravel()[i], want.ravel()[i]))


def slots_of(plan, M_dev):
    return [from_dev(plan.slot(M_dev, l)) for l in range(plan.n_layers)]


def check_superposition(plan, M_dev, M_ref, what="M", slots=None):
    for l in (range(plan.n_layers) if slots is None else slots):
        assert_bits_equal(from_dev(plan.slot(M_dev, l)), M_ref[l], "%s slot %d" % (what, l))


def check_model(out_dev, out_ref, what="out", positions=None):
    for l in (range(len(out_ref)) if positions is None else positions):
        assert_bits_equal(from_dev(out_dev[l]), out_ref[l], "%s layer %d" % (what, l))


def poison(t):
    """Fill a tensor with a NaN pattern so that unwritten elements are caught."""
    import torch

    if t.dtype == torch.bfloat16:
        t.view(torch.int16).fill_(-1)
    else:
        t.view(torch.int32).fill_(-1)
    return t
