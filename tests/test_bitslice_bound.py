"""The arithmetic behind the tolerance of the tensor-core MXFP4 path (no GPU): activations are written as a sum of six
block-scaled e2m1 terms, term i being the e2m1 rounding of what the earlier terms left over under the smallest power of
two that brings the leftover's largest magnitude to <= 6.  This file restates that rule in numpy and checks the error
bound the design derives from it (each term removes at least a factor 3 of a block's largest leftover), on random
blocks, on blocks with one outlier and on blocks at the ends of the float range."""
import numpy as np
import pytest

E2M1 = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])


def _round_e2m1(v):
    """Nearest e2m1 magnitude of |v| <= 6 (ties to either neighbour are both within the bound), with the sign."""
    idx = np.abs(np.abs(v)[..., None] - E2M1).argmin(axis=-1)
    return np.sign(v) * E2M1[idx]


def _slice(block, terms=6):
    """block: float64 [..., 32].  Returns the sum of the terms and the per-term largest leftovers."""
    r = block.astype(np.float64).copy()
    total = np.zeros_like(r)
    maxima = []
    for _ in range(terms):
        m = np.abs(r).max(axis=-1, keepdims=True)
        maxima.append(m[..., 0].copy())
        with np.errstate(divide="ignore"):
            ex = np.where(m > 0, np.ceil(np.log2(np.where(m > 0, m, 1.0) / 6.0)), 0.0)
        scale = np.exp2(np.clip(ex, -126, 126))
        q = _round_e2m1(np.clip(r / scale, -6.0, 6.0)) * scale
        total += q
        r = r - q
    maxima.append(np.abs(r).max(axis=-1))
    return total, np.stack(maxima)


@pytest.mark.parametrize("kind", ["normal", "outlier", "tiny", "huge", "sparse"])
def test_six_terms_leave_at_most_3_to_the_minus_6_of_the_block_maximum(kind):
    rng = np.random.default_rng(11)
    x = rng.standard_normal((2000, 32))
    if kind == "outlier":
        x[:, 5] *= 1000.0
    elif kind == "tiny":
        x *= 2.0 ** -100
    elif kind == "huge":
        x *= 2.0 ** 100
    elif kind == "sparse":
        x[rng.random(x.shape) < 0.8] = 0.0
    # bf16 inputs, as the kernels see them
    x = (x.astype(np.float32).view(np.uint32) & 0xFFFF0000).view(np.float32).astype(np.float64)
    total, maxima = _slice(x)
    m0 = maxima[0]
    nz = m0 > 0
    # every term removes at least a factor 3 of the largest leftover ...
    for i in range(6):
        assert np.all(maxima[i + 1][nz] <= maxima[i][nz] / 3.0 * (1 + 1e-12))
    # ... so the element error is at most 3^-6 of the block's largest magnitude
    err = np.abs(total - x).max(axis=-1)
    assert np.all(err[nz] <= m0[nz] * 3.0 ** -6 * (1 + 1e-12))
    assert np.all(total[~nz] == 0)


def test_sliced_dot_products_are_within_the_layer_tolerance():
    """The relative error of a long dot product with sliced activations is far below the 1e-2 of the parity tests."""
    rng = np.random.default_rng(12)
    x = rng.standard_normal((64, 7168))
    w = rng.standard_normal((7168, 16))
    xs = _slice(x.reshape(64, -1, 32))[0].reshape(64, 7168)
    ref, got = x @ w, xs @ w
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 2e-3
