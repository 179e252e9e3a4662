"""tq_fused_gemv_host_static: the host-operand GEMV for callers that must not allocate device
memory (inside a serving loop or a capture, where cudaMalloc would synchronise the device; in a
plug-in that owns no memory pool).  Its staging copies live in an array built into the library,
so the test checks that it gives what tq_fused_gemv_host gives with caller-allocated staging, on
two calls in a row (the array keeps the previous call's contents), and that it refuses sizes its
array cannot hold.  Collected last on purpose: a failure here cannot mask another test."""
import numpy as np
import pytest
import torch

from inputs import synth
from oracle import oracle

pytestmark = pytest.mark.gpu
TOL = 2e-3


def _matrix(tq, rows, cols, seed):
    rng = np.random.default_rng(seed)
    q = np.clip(np.rint(rng.standard_t(5, size=(rows, cols)) * 4), -127, 127).astype(np.int8)
    s = (rng.random(rows) + 0.5).astype(np.float32)
    d = oracle.Dictionary.build([q], top_k=3000)
    stream = d.encode(q)[0]
    dd = tq.tq_dict_upload(tq.tq_dict_from_entries(d.entries))
    return q, s, tq.tq_upload(dd, stream, rows, cols, s, None, levels_signed=True, layout=tq.TQ_LAYOUT_PLANES)


def test_static_staging_matches_caller_staging_twice():
    from paper_2509_22951_b200 import binding as tq

    rows, cols = 300, 2048
    q, s, m = _matrix(tq, rows, cols, 21)
    for call, B in enumerate((3, 1)):  # the second call reuses the array the first one filled
        x = synth.activations(B, cols, 40 + call).pin_memory()
        y_static = torch.full((B, rows), float("nan"), dtype=torch.float32).pin_memory()
        y_caller = torch.full((B, rows), float("nan"), dtype=torch.float32).pin_memory()
        tq.tq_fused_gemv_host_static(m, x, y_static)
        torch.cuda.synchronize()
        xs = torch.empty(B * cols, dtype=torch.bfloat16, device="cuda")
        ys = torch.empty(B * rows, dtype=torch.float32, device="cuda")
        tq.tq_fused_gemv_host(m, x, y_caller, xs, ys)
        torch.cuda.synchronize()
        a, b = y_static.numpy().astype(np.float64), y_caller.numpy().astype(np.float64)
        assert np.all(np.isfinite(a))
        err = np.max(np.max(np.abs(a - b), axis=1) / np.max(np.abs(b), axis=1))
        assert err <= TOL, err
        ref = oracle.layer_forward(q, s, x.double().numpy())
        assert np.max(np.max(np.abs(a - ref), axis=1) / np.max(np.abs(ref), axis=1)) <= TOL
    assert tq.tq_device_status(m) == 0


def test_static_staging_rejects_oversize():
    from paper_2509_22951_b200 import binding as tq

    rows, cols = 16, 16384  # 32 * 16384 elements of x do not fit the built-in array
    _, _, m = _matrix(tq, rows, cols, 22)
    x = synth.activations(32, cols, 50).pin_memory()
    y = torch.zeros((32, rows), dtype=torch.float32).pin_memory()
    with pytest.raises(tq.TqError) as e:
        tq.tq_fused_gemv_host_static(m, x, y)
    assert e.value.status == tq.TQ_ERR_UNSUPPORTED_SHAPE
    assert "262144" in str(e.value)
