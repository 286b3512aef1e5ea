"""The error bound behind the retrieval screen (host arithmetic only, no GPU).

The screening kernel rounds queries and unit-length candidates to bf16 and dismisses a candidate only
if its screened cosine is more than 8.5e-3 below the query's cut.  That is safe if the screened cosine
is never more than 8.5e-3 away from the exact one.  The bound: rounding to nearest with 8 significant
bits (bf16: 7 stored, one implied) changes a value by at most 2^-8 of itself, so a product by at most
(2^-7 + 2^-16) of itself, and by Cauchy-Schwarz the cosine by at most 2^-7 + 2^-16 = 7.83e-3.  Checked
here on random rows and on rows built so that every rounding error has the same sign and nearly the
largest size."""
import os
import re

import numpy as np

BOUND = 2.0 ** -7 + 2.0 ** -16
MARGIN = 8.5e-3          # kScreenEps of the kernel


def to_bf16(x):
    """fp32 -> nearest bf16 (ties to even), returned as fp32."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def screened_and_exact(q, c):
    """cosines of query rows q with candidate rows c: from bf16-rounded queries and bf16-rounded unit candidates, and exact."""
    q64, c64 = q.astype(np.float64), c.astype(np.float64)
    qn, cn = np.linalg.norm(q64, axis=1), np.linalg.norm(c64, axis=1)
    exact = (q64 @ c64.T) / np.outer(qn, cn)
    unit = (c64 / cn[:, None]).astype(np.float32)
    screened = (to_bf16(q).astype(np.float64) @ to_bf16(unit).astype(np.float64).T) / qn[:, None]
    return screened, exact


def test_bf16_rounding_is_within_half_a_unit():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(size=100_000), rng.normal(size=1000) * 1e-20, rng.normal(size=1000) * 1e20]).astype(np.float32)
    r = to_bf16(x)
    assert np.all(np.abs(r.astype(np.float64) - x.astype(np.float64)) <= 2.0 ** -8 * np.abs(x.astype(np.float64)))
    assert np.all((r.view(np.uint32) & 0xFFFF) == 0)


def test_screened_cosine_within_bound_on_random_rows():
    rng = np.random.default_rng(1)
    for d in (4, 64, 300, 1000):
        q = rng.normal(size=(64, d)).astype(np.float32)
        c = rng.normal(size=(512, d)).astype(np.float32) * rng.uniform(0.1, 10.0, size=(512, 1)).astype(np.float32)
        s, e = screened_and_exact(q, c)
        assert np.abs(s - e).max() <= BOUND < MARGIN
        # random rounding errors cancel in long rows (not in rows of 4 columns: 4.9e-3 is seen there)
        assert d < 300 or np.abs(s - e).max() < 1e-3


def test_screened_cosine_within_bound_when_every_rounding_error_points_the_same_way():
    # components just beside a rounding midpoint are all moved by almost 2^-8 of themselves; with query
    # and candidate parallel every product errs in the same direction
    d = 300
    below_mid = np.float32(1.0 + 2.0 ** -8 - 2.0 ** -20)          # rounds down to 1.0
    above_mid = np.float32(1.0 + 2.0 ** -8 + 2.0 ** -20)          # rounds up to 1 + 2^-7
    for val in (below_mid, above_mid):
        q = np.full((1, d), val, dtype=np.float32)
        c = np.full((1, d), val, dtype=np.float32) * np.float32(3.0)
        s, e = screened_and_exact(q, c)
        assert abs(e[0, 0] - 1.0) < 1e-12
        assert 1e-3 < abs(s[0, 0] - e[0, 0]) <= BOUND < MARGIN
    # opposite vectors: the error must not exceed the bound on the negative side either
    q = np.full((1, d), below_mid, dtype=np.float32)
    s, e = screened_and_exact(q, -q)
    assert abs(s[0, 0] - e[0, 0]) <= BOUND


def test_margin_covers_bound_and_fp32_accumulation():
    # fp32 accumulation of d = 1024 products of magnitude <= 1 and the two scalings add at most about
    # (d/16 + 4) 2^-24 to the bound (one rounding per 16-column MMA step plus the scalings)
    assert BOUND + (1024 / 16 + 4) * 2.0 ** -24 < MARGIN


def test_margin_is_the_kernels():
    src = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "paper_1606_08495_b200", "csrc",
                       "w2v_topk_tc.cu")
    with open(src) as f:
        m = re.search(r"constexpr float kScreenEps = ([0-9.eE+-]+)f;", f.read())
    assert m and float(m.group(1)) == MARGIN
