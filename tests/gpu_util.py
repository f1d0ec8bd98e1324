"""Helpers for the GPU parity tests: move oracle tensors to the device, compare within the stated bars."""
import numpy as np
import torch

from paper_2310_17723_b200 import hero

TORCH_FP = {"f16": torch.float16, "bf16": torch.bfloat16}


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def f32(a):
    return dev(np.asarray(a, np.float32))


def qt_to_device(qt):
    """Oracle QT -> (torch tensor, hero.Tensor).  INT8: payload + its scale; FP: cast to the storage type
    (exact: the oracle already rounded the values to that grid)."""
    if qt.kind == "fp":
        t = dev(qt.data, TORCH_FP[qt.dtype])
        return t, hero.tensor(t), None
    t = dev(qt.data)
    if qt.row_scale is not None:
        s = f32(qt.row_scale)
        return t, hero.tensor(t, "twq", s), s
    if qt.col_scale is not None:
        cs = np.asarray(qt.col_scale)
        if np.all(cs == cs[0]):                      # a static scale travels as one value (Eq. 5)
            s = f32(cs[:1])
            return t, hero.tensor(t, "sq", s), s
        s = f32(cs)
        return t, hero.tensor(t, "fwq", s), s
    return t, hero.tensor(t, "none"), None


def int8_mismatch(got, want):
    """(fraction of elements that differ, max abs difference) between two INT8 arrays."""
    g = np.asarray(got).astype(np.int32)
    w = np.asarray(want).astype(np.int32)
    d = np.abs(g - w)
    return float(np.mean(d != 0)), int(d.max()) if d.size else 0


def assert_int8_close(got, want, frac=1e-4, what=""):
    """The INT8 bar: bit-exact except at most 1 LSB on at most `frac` of the elements."""
    f, m = int8_mismatch(got, want)
    assert m <= 1, "%s: max INT8 difference %d LSB" % (what, m)
    # small tensors: allow a single tie
    assert f <= max(frac, 1.0 / max(np.asarray(want).size, 1)), "%s: %.3g of elements differ" % (what, f)


def rel_err(got, want):
    """max |g - o| / max |o| over the tensor."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    den = np.max(np.abs(want))
    return float(np.max(np.abs(got - want)) / (den if den > 0 else 1.0))
