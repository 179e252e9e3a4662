"""Domain of the integer tensor-core GEMV (TQ_LAYOUT_TILES): activation vectors far from N(0, 1).

The kernels put each bf16 activation vector on a fixed-point grid 30 bits below the power of two
above its largest magnitude, X = round(x * 2^(30 - e)) with max |x| < 2^e, and sum exact integers.
The only deviation from the exact product is that rounding, at most 2^(e - 31) per element, so for
every row
    |y - y_exact| <= scale_r * 2^(e - 31) * sum_c |q[r][c] - zero_r|  +  one fp32 rounding of y.
These tests check that bound element by element against the fp64 oracle for vectors with one huge
element, tiny (smallest-normal and subnormal) elements, all zeros, and the documented behaviour for
Inf / NaN (that vector's outputs are NaN, the others' are untouched, the status word stays 0),
through the single-matrix call and the stack, for 1, 2 and 8 vectors (the narrow and the wide kernel).
"""
import numpy as np
import pytest
import torch

from inputs import synth
from oracle import oracle

pytestmark = pytest.mark.gpu
CONTRACT = 2e-3  # max_r |y - y_ref| <= CONTRACT * max_r |y_ref| per vector
ROWS, COLS = 208, 3072


@pytest.fixture(scope="module")
def tq():
    from paper_2509_22951_b200 import binding
    return binding


@pytest.fixture(scope="module")
def layer(tq):
    """Signed levels, random scales; column 77 is the one the huge activation element sits on."""
    rng = np.random.default_rng(2024)
    q = np.clip(np.rint(rng.standard_t(5, size=(ROWS, COLS)) * 6), -127, 127).astype(np.int8)
    s = (rng.random(ROWS) + 0.5).astype(np.float32)
    out = {}
    for name, qq in (("dense", q), ("zero_column", np.where(np.arange(COLS)[None, :] == 77, 0, q).astype(np.int8))):
        d = oracle.Dictionary.build([qq])
        stream = d.encode(qq)[0]
        dd = tq.tq_dict_upload(tq.tq_dict_from_entries(d.entries))
        out[name] = (qq, s, tq.tq_upload(dd, stream, ROWS, COLS, s, layout=tq.TQ_LAYOUT_TILES))
    return out


def _bf16(a):
    return torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)


def _run_both(tq, m, x):
    """y through tq_fused_gemv and through a one-matrix stack; they must agree bit for bit."""
    xd = x.cuda()
    y1 = tq.tq_fused_gemv(m, xd)
    y2 = torch.full_like(y1, float("nan"))
    tq.tq_fused_gemv_stack(tq.tq_stack_create([m], [xd], [y2]))
    torch.cuda.synchronize()
    assert torch.equal(y1, y2) or (torch.isnan(y1) == torch.isnan(y2)).all() and torch.equal(torch.nan_to_num(y1), torch.nan_to_num(y2))
    return y1.cpu().numpy().astype(np.float64)


def _bound(q, s, x):
    """The documented bound per (vector, row): grid rounding plus one fp32 rounding of the result."""
    xa = np.abs(x.double().numpy())
    e = np.floor(np.log2(np.maximum(xa.max(axis=1), 2.0 ** -126))) + 1  # max |x| < 2^e, e >= -126
    l1 = np.abs(q.astype(np.float64)).sum(axis=1) * s.astype(np.float64)
    return (2.0 ** (e - 31))[:, None] * l1[None, :]


def _check(tq, layer, which, x, contract=True):
    q, s, m = layer[which]
    y = _run_both(tq, m, x)
    ref = oracle.layer_forward(q, s, x.double().numpy())
    assert np.all(np.isfinite(y))
    slack = np.abs(ref) * 2.0 ** -23 + 2.0 ** -149  # fp32 rounding of the output (subnormal results included)
    assert np.all(np.abs(y - ref) <= _bound(q, s, x) + slack)
    rel = np.max(np.abs(y - ref), axis=1) / np.maximum(np.max(np.abs(ref), axis=1), 1e-300)
    if contract:
        assert float(rel.max()) <= CONTRACT, rel
    assert tq.tq_device_status(m) == 0
    return float(rel.max())


@pytest.mark.parametrize("B", [1, 2, 8])
def test_all_zero_vector(tq, layer, B):
    q, s, m = layer["dense"]
    x = synth.activations(B, COLS, 11)
    x[B - 1] = 0
    y = _run_both(tq, m, x)
    assert np.all(y[B - 1] == 0.0)
    if B > 1:
        ref = oracle.layer_forward(q, s, x.double().numpy())
        assert np.max(np.abs(y[0] - ref[0])) <= 1e-6 * np.max(np.abs(ref[0]))


@pytest.mark.parametrize("B", [1, 2, 8])
@pytest.mark.parametrize("which", ["dense", "zero_column"])
@pytest.mark.parametrize("log2_big", [12, 20])
def test_one_huge_element(tq, layer, B, which, log2_big):
    """One element 2^12 or 2^20 times the others.  Under random weights it dominates y and the other
    elements' rounding is invisible; with zero weights under it the result rests on the small
    elements alone, which still keep 30 - 3 - log2_big bits below N(0, 1)'s largest values."""
    x = synth.activations(B, COLS, 20 + B).float()
    x[:, 77] = 2.0 ** log2_big * (1.0 + 0.25 * torch.arange(B))
    rel = _check(tq, layer, which, _bf16(x.numpy()))
    if log2_big == 12 or which == "dense":
        assert rel <= 1e-5


@pytest.mark.parametrize("B", [1, 2, 8])
def test_beyond_the_grid_the_bound_still_holds(tq, layer, B):
    """An element 2^36 times the rest with zero weights under it: the rest falls below the 30-bit grid,
    the 2e-3 contract no longer applies, the stated bound does."""
    x = synth.activations(B, COLS, 30 + B).float()
    x[:, 77] = 2.0 ** 36
    _check(tq, layer, "zero_column", _bf16(x.numpy()), contract=False)


@pytest.mark.parametrize("B", [1, 2, 8])
def test_tiny_and_subnormal_vectors(tq, layer, B):
    """Vectors near the bottom of the bf16 range: smallest normal values (2^-126 scale) and pure
    subnormals (multiples of 2^-133).  The grid reaches 2^-156, so both are exact."""
    g = synth.activations(B, COLS, 40 + B).float().numpy()
    tiny = g * 2.0 ** -126  # normal and subnormal bf16 values mixed
    rel = _check(tq, layer, "dense", _bf16(tiny))
    assert rel <= 1e-5
    if B > 1:
        sub = np.rint(g * 20.0) * 2.0 ** -133  # subnormals only, integers times the bf16 quantum
        sub = np.clip(sub, -127 * 2.0 ** -133, 127 * 2.0 ** -133)
        xs = torch.from_numpy(sub.astype(np.float32)).to(torch.bfloat16)
        assert float(xs.float().abs().max()) < 2.0 ** -126
        rel = _check(tq, layer, "dense", xs)
        assert rel <= 1e-5


@pytest.mark.parametrize("B", [1, 2, 8])
def test_largest_finite_values(tq, layer, B):
    x = synth.activations(B, COLS, 50 + B).float()
    x = x / x.abs().max() * 3.0e38
    q, s, m = layer["dense"]
    xb = _bf16(x.numpy())
    assert torch.isfinite(xb.float()).all()
    y = _run_both(tq, m, xb)
    ref = oracle.layer_forward(q, s, xb.double().numpy())
    ok = np.abs(ref) < 3.0e38  # results beyond fp32 become Inf on both sides
    assert np.all(np.abs(y - ref)[ok] <= _bound(q, s, xb)[ok] + np.abs(ref[ok]) * 2.0 ** -23)
    assert np.all(np.isinf(y[~ok]) | (np.abs(y[~ok]) > 3.0e38))


@pytest.mark.parametrize("B", [1, 2, 8])
@pytest.mark.parametrize("bad", [float("inf"), float("-inf"), float("nan")])
def test_non_finite_element_gives_nan_for_that_vector_only(tq, layer, B, bad):
    q, s, m = layer["dense"]
    x = synth.activations(B, COLS, 60 + B)
    x[B - 1, 5] = bad
    y = _run_both(tq, m, x)
    assert np.all(np.isnan(y[B - 1]))
    if B > 1:
        ref = oracle.layer_forward(q, s, x[: B - 1].double().numpy())
        assert np.all(np.isfinite(y[: B - 1]))
        assert np.max(np.abs(y[: B - 1] - ref)) <= 1e-6 * np.max(np.abs(ref))
    assert tq.tq_device_status(m) == 0
