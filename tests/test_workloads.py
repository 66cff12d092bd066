"""Seeded input generator and workload definitions (no GPU needed)."""
import json
import os

import numpy as np
import pytest

import workloads
from workloads import hashgen
from workloads.configs import ALIGN_ELEMS, Layout, draw_log_uniform_sizes

M1, M2, M3, M4 = 0x6a09e667f3bcc909, 0xbb67ae8584caa73b, 0x3c6ef372fe94f82b, 0xa54ff53a5f1d36f1
MASK = (1 << 64) - 1


def py_mix(x):
    x ^= x >> 32
    x = (x * M1) & MASK
    x ^= x >> 29
    x = (x * M2) & MASK
    x ^= x >> 32
    return x


def py_hash(seed, stream, step, worker, idx):
    key = py_mix((seed + M3) & MASK)
    ctr = (stream << 60) | (step << 40) | (worker << 32) | idx
    return py_mix((py_mix(ctr ^ key) + M4) & MASK)


# known answers of the hash, (seed, stream, step, worker, idx) -> h
KNOWN = {
    (1, 0, 0, 0, 0): 0xcb844baeeca499f6,
    (1, 0, 0, 0, 1): 0x20d827488547beb1,
    (1, 0, 9, 3, 1048575): 0x19ace05c6b89ff20,
    (2, 0, 49, 7, 11699999): 0x80d631f9f9efac1a,
    (5, 1, 29, 15, 29999): 0xeb8cb9decb55f860,
    (1, 2, 0, 0, 0): 0x2c0fe344dfb67a43,
    (3, 3, 0, 0, 160): 0x71723a36b97e4485,
}


def test_constants_are_square_root_fractions():
    from decimal import Decimal, getcontext
    getcontext().prec = 60
    for prime, const in ((2, M1), (3, M2), (5, M3), (7, M4)):
        frac = Decimal(prime).sqrt() % 1
        assert int(frac * (1 << 64)) | 1 == const


def test_hash_known_answers():
    for args, want in KNOWN.items():
        assert hashgen.hash64(*args) == want
        assert py_hash(*args) == want


def test_uniform_and_init_values():
    idx = np.array([0, 1, 5, 1048575], dtype=np.int64)
    got = hashgen.grad_uniform(1, 9, 3, idx=idx, scale=1e-2)
    for k, j in enumerate(idx):
        u24 = py_hash(1, 0, 9, 3, int(j)) >> 40
        want = np.float32(1e-2) * np.float32((u24 - 2 ** 23) * 2.0 ** -23)
        assert got[k] == want
    w = hashgen.init_global(1, idx0=0, n=4)
    for j in range(4):
        u24 = py_hash(1, 2, 0, 0, j) >> 40
        assert w[j] == np.float32(0.1) * np.float32((u24 - 2 ** 23) * 2.0 ** -23)
    # range and index-list forms agree
    np.testing.assert_array_equal(hashgen.grad_uniform(1, 2, 1, idx0=10, n=50),
                                  hashgen.grad_uniform(1, 2, 1, idx=np.arange(10, 60)))


def test_gaussian_definition_and_moments():
    import math
    g = hashgen.grad_gauss(2, 3, 1, idx0=0, n=8, sigma=1e-3)
    for j in range(8):
        h = py_hash(2, 0, 3, 1, j)
        u1 = ((h >> 40) + 1) * 2.0 ** -24
        t = ((h >> 16) & 0xFFFFFF) * 2.0 ** -24
        z = math.sqrt(-2.0 * math.log(u1)) * math.cos(2 * math.pi * t)
        assert abs(g[j] - np.float32(1e-3 * z)) <= abs(np.spacing(np.float32(1e-3 * z)))
    z = hashgen.grad_gauss(2, 0, 0, idx0=0, n=200_000, sigma=1.0).astype(np.float64)
    assert abs(z.mean()) < 0.01
    assert abs(z.var() - 1.0) < 0.01
    assert abs((z ** 4).mean() - 3.0) < 0.08
    assert np.abs(z).max() <= 5.77
    u = hashgen.grad_uniform(1, 0, 0, idx0=0, n=200_000, scale=1.0).astype(np.float64)
    assert abs(u.mean()) < 0.01 and abs(u.var() - 1 / 3) < 0.005
    # neighbouring indices, workers and steps are uncorrelated
    a = hashgen.grad_uniform(1, 0, 0, idx0=0, n=200_000, scale=1.0)
    for b in (hashgen.grad_uniform(1, 0, 1, idx0=0, n=200_000, scale=1.0),
              hashgen.grad_uniform(1, 1, 0, idx0=0, n=200_000, scale=1.0),
              np.roll(a, 1)):
        assert abs(np.corrcoef(a, b)[0, 1]) < 0.01


def test_row_mask_rate():
    cfg = workloads.get("cfg5")
    rows = cfg.sparse_rows(0, 0)
    assert len(rows) == 2882                       # ~10 % of 30,000 rows
    assert np.all(np.diff(rows) > 0)
    assert not np.array_equal(rows, cfg.sparse_rows(1, 0))


def test_bf16_round_trip():
    x = np.array([1.0, 1.00390625, 1.01171875, -3.1415927, 1e-3, 0.0], dtype=np.float32)
    bits = hashgen.f32_to_bf16(x)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7: nearest even keeps 1.0;
    # 1 + 3*2^-8 is a tie between 1 + 2^-7 and 1 + 2^-6: nearest even takes 1 + 2^-6
    assert bits[0] == 0x3F80 and bits[1] == 0x3F80 and bits[2] == 0x3F82
    back = hashgen.bf16_to_f32(bits)
    assert np.all(np.abs(back - x) <= np.abs(x) * 2.0 ** -8)
    import torch
    want = torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits, want)


@pytest.mark.parametrize("name,K,P,n", [("cfg1", 4, 1_048_576, 1), ("cfg2", 8, 11_700_000, 62),
                                        ("cfg3", 8, 25_600_000, 161), ("cfg4", 16, 138_000_000, 32),
                                        ("cfg5", 16, 78_789_936, 15)])
def test_workload_shapes(name, K, P, n):
    cfg = workloads.get(name)
    assert (cfg.K, cfg.P, len(cfg.sizes)) == (K, P, n)
    lay = cfg.layout
    assert all(o % ALIGN_ELEMS == 0 for o in lay.offsets)
    assert lay.P_pad >= P and lay.P_pad % ALIGN_ELEMS == 0
    if name in ("cfg2", "cfg3"):
        assert min(cfg.sizes) >= 64 and max(cfg.sizes) <= 2_400_000
    if name == "cfg4":
        assert cfg.sizes[:3] == (102_760_448, 16_777_216, 4_096_000)


def test_committed_layouts_match_the_generator():
    here = os.path.dirname(workloads.__file__)
    for name, seed, n, total, first in (("cfg2", 2, 62, 11_700_000, 0), ("cfg3", 3, 161, 25_600_000, 0),
                                        ("cfg4", 4, 29, 14_366_336, 3)):
        sizes = json.load(open(os.path.join(here, "layouts", name + ".json")))["sizes"]
        assert sizes[-n:] == draw_log_uniform_sizes(seed, n, total, first_tensor=first)


def test_layout_pack_unpack():
    lay = Layout([5, 64, 33, 1])
    assert lay.offsets == [0, 32, 96, 160] and lay.P_pad == 192 and lay.P == 103
    flat = np.arange(1, 104, dtype=np.float32)
    padded = lay.pack(flat)
    np.testing.assert_array_equal(lay.unpack(padded), flat)
    assert padded[5:32].sum() == 0
    idx = np.array([0, 4, 5, 68, 69, 102])
    np.testing.assert_array_equal(padded[lay.padded_index(idx)], flat[idx])


def test_sparse_gradient_is_dense_with_zero_rows():
    cfg = workloads.get("cfg5").subset("mini", [40 * 8, 100, 7], sparse=(0, 40, 8))
    g = cfg.gradient(3, 2)
    rows = cfg.sparse_rows(3, 2)
    seg = g[:320].reshape(40, 8)
    mask = np.zeros(40, bool)
    mask[rows] = True
    assert np.all(seg[~mask] == 0) and np.all(seg[mask] != 0)
    idx = np.array([0, 9, 17, 319, 320, 426])
    np.testing.assert_array_equal(cfg.gradient(3, 2, idx), g[idx])
