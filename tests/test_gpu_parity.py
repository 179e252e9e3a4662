"""CUDA path against the oracle, through the C ABI.  Decoded bytes must be bit-exact; layer
outputs must satisfy max_r |y - y_ref| <= 2e-3 * max_r |y_ref| per batch column (the contract),
and the fused GEMV calls are held to the 1e-5 they deliver on N(0, 1) activations."""
import numpy as np
import pytest
import torch

from inputs import synth
from oracle import oracle

pytestmark = pytest.mark.gpu
TOL = 2e-3    # the contract: max_r |y - y_ref| <= TOL * max_r |y_ref| per vector
TIGHT = 1e-5  # what the GEMV kernels deliver on N(0, 1) activations (exact products; integer sums in the
              # tiles layout, fp32 sums in the others): a defect a hundred times smaller than TOL fails
GEMM_TIGHT = 5e-5  # the tensor-core products: exact bf16 operands, fp32 accumulation over up to 8192 columns


@pytest.fixture(scope="module")
def tq():
    from paper_2509_22951_b200 import binding
    return binding


LAYOUTS = [0, 1, 2]  # TQ_LAYOUT_STREAM, TQ_LAYOUT_PLANES, TQ_LAYOUT_TILES


@pytest.fixture(params=LAYOUTS, ids=["stream", "planes", "tiles"])
def layout(request):
    return request.param


def _rel_err(y, ref):
    # per batch column
    return float(np.max(np.max(np.abs(y - ref), axis=1) / np.max(np.abs(ref), axis=1)))


def _oracle_pack(q_list, top_k=65535):
    d = oracle.Dictionary.build(q_list, top_k=top_k)
    return d, [d.encode(q)[0] for q in q_list]


def _upload_from_oracle(tq, odict, stream, rows, cols, scale, zero=None, signed=True, layout=0):
    """Everything fed to the device comes from the oracle (table, stream) so a host-library bug
    cannot hide a device bug."""
    hd = tq.tq_dict_from_entries(odict.entries)
    dd = tq.tq_dict_upload(hd)
    return tq.tq_upload(dd, stream, rows, cols, scale, zero, levels_signed=signed, layout=layout)


def _check_layer(tq, q, scale, odict, stream, batches=(1,), zero=None, seed=1, layout=0):
    rows, cols = q.shape
    m = _upload_from_oracle(tq, odict, stream, rows, cols, scale, zero, signed=(q.dtype == np.int8), layout=layout)
    # decoded bytes: bit exact against the oracle's decoder and the original levels
    got = tq.tq_decompress(m).cpu().numpy()
    ref = odict.decode(stream).reshape(rows, cols)
    assert np.array_equal(ref, q.view(np.uint8))
    assert np.array_equal(got, ref)
    for B in batches:
        x = synth.activations(B, cols, seed + B)
        y = tq.tq_fused_gemv(m, x.cuda()).cpu().numpy().astype(np.float64)
        yref = oracle.layer_forward(q, scale, x.double().numpy(), zero=zero)
        assert y.shape == yref.shape
        assert _rel_err(y, yref) <= TIGHT
    assert tq.tq_device_status(m) == 0
    return m


def test_config0_layer_2048x2048(tq, layout):
    w = synth.weight(2048, 2048, synth.matrix_seed(0)).numpy()
    q, s = oracle.quantize_rows(w)
    d, (stream,) = _oracle_pack([q])
    m = _check_layer(tq, q, s, d, stream, batches=(1, 4), layout=layout)
    assert m.info.n_hits + m.info.n_miss == 2048 * 2048 // 4
    assert m.info.stream_bytes == stream.nbytes


@pytest.mark.parametrize("rows,cols", [(1, 4), (3, 8), (7, 260), (8, 256), (9, 1028), (33, 2052), (17, 8192), (5, 12288),
                                       (40, 4 * 300), (35, 28672)])
def test_ragged_shapes(tq, rows, cols, layout):
    if layout == 2 and cols > tq.TQ_TILES_MAX_COLS:
        with pytest.raises(tq.TqError) as e:
            tq.tq_upload_size(np.zeros(rows * cols // 4, dtype=np.uint16) + 1, rows, cols, layout)
        assert e.value.status == tq.TQ_ERR_UNSUPPORTED_SHAPE
        return
    rng = np.random.default_rng(rows * 1000 + cols)
    q = np.clip(np.rint(rng.standard_t(5, size=(rows, cols)) * 3), -127, 127).astype(np.int8)
    s = (rng.random(rows) + 0.5).astype(np.float32)
    d, (stream,) = _oracle_pack([q], top_k=200)
    _check_layer(tq, q, s, d, stream, batches=(1, 2, 3, 4, 5), layout=layout)


def test_all_hits_and_all_misses(tq, layout):
    rng = np.random.default_rng(5)
    q = rng.integers(-2, 3, size=(64, 512)).astype(np.int8)
    s = np.full(64, 0.01, dtype=np.float32)
    d, (stream,) = _oracle_pack([q])
    assert np.all(stream != 0xFFFF)  # every group is in the table
    _check_layer(tq, q, s, d, stream, batches=(1, 4), layout=layout)
    d0, (stream0,) = _oracle_pack([q], top_k=0)
    assert stream0.size == 5 * q.size // 4  # every group escapes
    _check_layer(tq, q, s, d0, stream0, batches=(1, 3), layout=layout)


def test_large_table_codes_near_65534(tq, layout):
    # enough distinct windows to fill the table; high codes (>= 0xFF00) share their top byte with the marker
    rng = np.random.default_rng(6)
    q = rng.integers(-20, 21, size=(512, 1024)).astype(np.int8)
    s = (rng.random(512) + 0.5).astype(np.float32)
    d, (stream,) = _oracle_pack([q])
    assert d.K == 65534 and int(stream[stream != 0xFFFF].max()) > 0xFF00
    _check_layer(tq, q, s, d, stream, batches=(1,), layout=layout)


def test_unsigned_levels_with_zero_point(tq, layout):
    # the paper's own quantizer: per-tensor unsigned levels and a zero point
    w = synth.weight(256, 1024, synth.matrix_seed(9)).numpy()
    qu, sc, zp = oracle.quantize_paper(w)
    qu = qu.reshape(256, 1024)
    s = np.full(256, sc, dtype=np.float32)
    z = np.full(256, zp, dtype=np.float32)
    d, (stream,) = _oracle_pack([qu])
    _check_layer(tq, qu, s, d, stream, batches=(1, 4), zero=z, layout=layout)


@pytest.mark.parametrize("bits", [6, 4, 2])
def test_lower_bit_grids_of_the_per_tensor_quantizer(tq, layout, bits):
    # Listing 1 at fewer bits: levels 0..2^bits-1 in one byte each; table, tokens, decode and products unchanged
    w = synth.weight(144, 1536, synth.matrix_seed(20 + bits)).numpy()
    qu, sc, zp = oracle.quantize_paper(w, bits=bits)
    qu = qu.reshape(144, 1536)
    assert int(qu.max()) == 2 ** bits - 1
    s = np.full(144, sc, dtype=np.float32)
    z = np.full(144, zp, dtype=np.float32)
    d, (stream,) = _oracle_pack([qu])
    _check_layer(tq, qu, s, d, stream, batches=(1, 3, 8), zero=z, layout=layout)


def test_batch_up_to_32(tq, layout):
    rng = np.random.default_rng(8)
    q = np.clip(np.rint(rng.standard_t(5, size=(130, 3072)) * 6), -127, 127).astype(np.int8)
    s = (rng.random(130) + 0.5).astype(np.float32)
    d, (stream,) = _oracle_pack([q])
    _check_layer(tq, q, s, d, stream, batches=(8, 32), layout=layout)


def test_quantize_rows_device_bit_exact(tq):
    w = synth.weight(300, 3072, synth.matrix_seed(11), device="cuda")
    w[17] = 0
    q, s = tq.tq_quantize_rows_device(w)
    qo, so = oracle.quantize_rows(w.cpu().numpy())
    assert np.array_equal(q.cpu().numpy(), qo) and np.array_equal(s.cpu().numpy(), so)


def test_generator_is_device_independent():
    a = synth.weight(64, 2048, synth.matrix_seed(2), device="cpu")
    b = synth.weight(64, 2048, synth.matrix_seed(2), device="cuda").cpu()
    assert torch.equal(a, b)
    xa = synth.activations(4, 2048, 5, device="cpu")
    xb = synth.activations(4, 2048, 5, device="cuda").cpu()
    assert torch.equal(xa, xb)


def test_host_library_pipeline_matches_oracle_pipeline(tq, layout):
    """Product pipeline end to end (tq_quantize_rows_device -> tq_build_dictionary -> tq_encode ->
    tq_upload -> kernels) on the 1B MLP shapes, checked on sampled rows the oracle computes itself."""
    shapes = [("gate", 8192, 2048), ("up", 8192, 2048), ("down", 2048, 8192)]
    ws = [synth.weight(r, c, synth.matrix_seed(100 + i), device="cuda") for i, (_, r, c) in enumerate(shapes)]
    qs, ss = zip(*[tq.tq_quantize_rows_device(w) for w in ws])
    q_host = [q.cpu().numpy() for q in qs]
    hd = tq.tq_build_dictionary(q_host)
    dd = tq.tq_dict_upload(hd)
    rng = np.random.default_rng(3)
    for i, (name, rows, cols) in enumerate(shapes):
        stream, h, mi = tq.tq_encode(hd, q_host[i])
        assert stream.size == h + 5 * mi
        m = tq.tq_upload(dd, stream, rows, cols, ss[i].cpu().numpy(), layout=layout)
        got = tq.tq_decompress(m)
        assert torch.equal(got.view(torch.int8), qs[i])  # whole matrix, product vs product
        sample = np.sort(rng.choice(rows, 64, replace=False))
        qo, so = oracle.quantize_rows(ws[i][sample].cpu().numpy())  # oracle quantizes the sampled rows itself
        assert np.array_equal(got[sample].cpu().numpy().view(np.int8), qo)
        for B in (1, 4):
            x = synth.activations(B, cols, 40 + i)
            y = tq.tq_fused_gemv(m, x.cuda()).cpu().numpy().astype(np.float64)
            yref = oracle.layer_forward(qo, so, x.double().numpy())
            err = np.max(np.abs(y[:, sample] - yref), axis=1) / np.max(np.abs(yref), axis=1)
            assert float(err.max()) <= TIGHT
        assert tq.tq_device_status(m) == 0


# ------------------------------------------------------------------ prefill product (tcgen05)
@pytest.mark.parametrize("rows,cols,M", [(128, 128, 256), (256, 512, 300), (130, 264, 1), (384, 3072, 2048), (100, 1024, 77)])
def test_fused_gemm_matches_oracle(tq, rows, cols, M):
    rng = np.random.default_rng(rows + cols + M)
    q = np.clip(np.rint(rng.standard_t(5, size=(rows, cols)) * 6), -127, 127).astype(np.int8)
    s = (rng.random(rows) + 0.5).astype(np.float32)
    d, (stream,) = _oracle_pack([q], top_k=3000)
    m = _upload_from_oracle(tq, d, stream, rows, cols, s, layout=1)
    X = synth.activations(M, cols, 123)
    Y = tq.tq_fused_gemm(m, X.cuda()).cpu().numpy().astype(np.float64)
    assert tq.tq_device_status(m) == 0
    sample = np.arange(M) if M <= 300 else np.sort(rng.choice(M, 64, replace=False))
    Yref = oracle.layer_forward(q, s, X[sample].double().numpy())
    assert Y.shape == (M, rows)
    assert _rel_err(Y[sample], Yref) <= GEMM_TIGHT


def test_fused_gemm_unsigned_levels_with_zero_point(tq):
    w = synth.weight(256, 512, synth.matrix_seed(21)).numpy()
    qu, sc, zp = oracle.quantize_paper(w)
    qu = qu.reshape(256, 512)
    s = np.full(256, sc, dtype=np.float32)
    z = np.full(256, zp, dtype=np.float32)
    d, (stream,) = _oracle_pack([qu])
    m = _upload_from_oracle(tq, d, stream, 256, 512, s, zero=z, signed=False, layout=1)
    X = synth.activations(64, 512, 9)
    Y = tq.tq_fused_gemm(m, X.cuda()).cpu().numpy().astype(np.float64)
    Yref = oracle.layer_forward(qu, s, X.double().numpy(), zero=z)
    assert _rel_err(Y, Yref) <= GEMM_TIGHT
    assert tq.tq_device_status(m) == 0


def test_fused_gemm_agrees_with_fused_gemv(tq):
    rng = np.random.default_rng(77)
    q = np.clip(np.rint(rng.standard_t(5, size=(512, 2048)) * 8), -127, 127).astype(np.int8)
    s = (rng.random(512) + 0.5).astype(np.float32)
    d, (stream,) = _oracle_pack([q])
    m = _upload_from_oracle(tq, d, stream, 512, 2048, s, layout=1)
    X = synth.activations(8, 2048, 5).cuda()
    a = tq.tq_fused_gemm(m, X)
    b = tq.tq_fused_gemv(m, X)
    assert float((a - b).abs().max() / b.abs().max()) < 1e-5


# ------------------------------------------------------------------ prefill product, two phases (TILES)
@pytest.mark.parametrize("rows,cols,M", [(128, 128, 256), (256, 512, 300), (130, 264, 1), (384, 3072, 2048),
                                         (100, 1024, 77), (1000, 8192, 513), (17, 8, 5)])
def test_fused_gemm_ws_matches_oracle(tq, rows, cols, M):
    """Decode once to bf16 in a workspace, then the TMA-fed tcgen05 GEMM: ragged rows, columns and
    token counts (tiles of 128 rows x 256 tokens x 64 columns), several tiles per CTA at M = 2048."""
    rng = np.random.default_rng(rows + cols + M)
    q = np.clip(np.rint(rng.standard_t(5, size=(rows, cols)) * 6), -127, 127).astype(np.int8)
    s = (rng.random(rows) + 0.5).astype(np.float32)
    d, (stream,) = _oracle_pack([q], top_k=3000)
    m = _upload_from_oracle(tq, d, stream, rows, cols, s, layout=2)
    ws = torch.full((tq.tq_gemm_workspace_size(m),), 0x7F, dtype=torch.uint8, device="cuda")  # NaN-ish garbage
    X = synth.activations(M, cols, 123)
    for _ in range(2):
        Y = tq.tq_fused_gemm_ws(m, X.cuda(), ws).cpu().numpy().astype(np.float64)
    assert tq.tq_device_status(m) == 0
    sample = np.arange(M) if M <= 300 else np.sort(rng.choice(M, 64, replace=False))
    Yref = oracle.layer_forward(q, s, X[sample].double().numpy())
    assert Y.shape == (M, rows)
    assert _rel_err(Y[sample], Yref) <= GEMM_TIGHT


def test_fused_gemm_ws_unsigned_levels_with_zero_point(tq):
    w = synth.weight(256, 512, synth.matrix_seed(21)).numpy()
    qu, sc, zp = oracle.quantize_paper(w)
    qu = qu.reshape(256, 512)
    s = np.full(256, sc, dtype=np.float32)
    z = np.full(256, zp, dtype=np.float32)
    d, (stream,) = _oracle_pack([qu])
    m = _upload_from_oracle(tq, d, stream, 256, 512, s, zero=z, signed=False, layout=2)
    ws = torch.empty(tq.tq_gemm_workspace_size(m), dtype=torch.uint8, device="cuda")
    X = synth.activations(64, 512, 9)
    Y = tq.tq_fused_gemm_ws(m, X.cuda(), ws).cpu().numpy().astype(np.float64)
    Yref = oracle.layer_forward(qu, s, X.double().numpy(), zero=z)
    assert _rel_err(Y, Yref) <= GEMM_TIGHT
    assert tq.tq_device_status(m) == 0


def test_fused_gemm_ws_agrees_with_fused_gemv(tq):
    rng = np.random.default_rng(78)
    q = np.clip(np.rint(rng.standard_t(5, size=(512, 2048)) * 8), -127, 127).astype(np.int8)
    s = (rng.random(512) + 0.5).astype(np.float32)
    d, (stream,) = _oracle_pack([q])
    m = _upload_from_oracle(tq, d, stream, 512, 2048, s, layout=2)
    ws = torch.empty(tq.tq_gemm_workspace_size(m), dtype=torch.uint8, device="cuda")
    X = synth.activations(8, 2048, 5).cuda()
    a = tq.tq_fused_gemm_ws(m, X, ws)
    b = tq.tq_fused_gemv(m, X)
    assert float((a - b).abs().max() / b.abs().max()) < 1e-5


@pytest.mark.parametrize("M", [5, 130, 600])
def test_gemm_plan_matches_oracle(tq, M):
    """Several workspace GEMMs in one persistent launch: matrices of different row and column counts
    (ragged in both), one table, tiles of all products in one sequence; run twice on the same plan."""
    shapes = [(200, 512), (128, 1032), (17, 8), (384, 3072), (130, 264)]
    rng = np.random.default_rng(900 + M)
    qs = [np.clip(np.rint(rng.standard_t(5, size=sh) * 6), -127, 127).astype(np.int8) for sh in shapes]
    ss = [(rng.random(sh[0]) + 0.5).astype(np.float32) for sh in shapes]
    d, streams = _oracle_pack(qs, top_k=3000)
    hd = tq.tq_dict_from_entries(d.entries)
    dd = tq.tq_dict_upload(hd)
    mats = [tq.tq_upload(dd, st, sh[0], sh[1], sc, None, levels_signed=True, layout=2) for st, sh, sc in zip(streams, shapes, ss)]
    wss = [torch.full((tq.tq_gemm_workspace_size(m),), 0x7F, dtype=torch.uint8, device="cuda") for m in mats]
    Xs = [synth.activations(M, sh[1], 50 + i) for i, sh in enumerate(shapes)]
    Xd = [x.cuda() for x in Xs]
    plan = tq.tq_gemm_plan_create(mats, Xd, wss)
    stack = tq.tq_stack_create(mats)
    tq.tq_decode_bf16_stack(stack, wss)
    for _ in range(2):
        for y in plan.Ys:
            y.fill_(float("nan"))
        tq.tq_gemm_plan_run(plan)
    assert tq.tq_gemm_plan_status(plan) == 0
    for q, sc, x, y, m in zip(qs, ss, Xs, plan.Ys, mats):
        Y = y.cpu().numpy().astype(np.float64)
        sample = np.arange(M) if M <= 300 else np.sort(rng.choice(M, 64, replace=False))
        Yref = oracle.layer_forward(q, sc, x[sample].double().numpy())
        assert Y.shape == (M, q.shape[0]) and np.isfinite(Y).all()
        assert _rel_err(Y[sample], Yref) <= GEMM_TIGHT
        # and bit for bit what the single-matrix call gives
        Y1 = tq.tq_gemm_bf16_ws(m, x.cuda(), wss[mats.index(m)])
        assert torch.equal(Y1, y)


# ------------------------------------------------------------------ device-side table build
@pytest.mark.parametrize("case", ["ties", "several", "minus_one", "odd_lengths", "top_k_small", "large"])
def test_build_dictionary_device_matches_oracle(tq, case):
    """Listing 2 with the counting on the GPU: entries (rank order: count descending, then first
    occurrence) and counts must equal the oracle's and the host builder's, ties included."""
    rng = np.random.default_rng(sum(map(ord, case)))
    top_k = 65535
    if case == "ties":  # few distinct values: many windows share a count
        mats = [rng.integers(-1, 2, size=(40, 64)).astype(np.int8)]
    elif case == "several":  # windows must not span two matrices
        mats = [rng.integers(-3, 4, size=s).astype(np.int8) for s in [(16, 32), (7, 12), (64, 128)]]
    elif case == "minus_one":  # the window 0xFFFFFFFF (four levels of -1) is an ordinary window
        a = rng.integers(-2, 1, size=(32, 256)).astype(np.int8)
        a[:, 64:192] = -1
        mats = [a]
    elif case == "odd_lengths":  # lengths that are no multiple of 4, and matrices too short for one window
        mats = [rng.integers(-2, 3, size=n).astype(np.int8) for n in (1001, 3, 4, 4099, 2)]
    elif case == "top_k_small":
        mats = [rng.integers(-4, 5, size=(128, 256)).astype(np.int8)]
        top_k = 37
    else:  # more distinct windows than table entries, realistic levels
        mats = [np.clip(np.rint(rng.standard_t(5, size=(1024, 1024)) * 6), -127, 127).astype(np.int8),
                np.clip(np.rint(rng.standard_t(5, size=(512, 2048)) * 9), -127, 127).astype(np.int8)]
    od = oracle.Dictionary.build(mats, top_k=top_k)
    hd = tq.tq_build_dictionary(mats, top_k=top_k)
    dev = [torch.from_numpy(np.ascontiguousarray(m).reshape(-1).view(np.uint8).copy()).cuda() for m in mats]
    # 4-byte alignment of every matrix is the call's requirement; torch allocations satisfy it
    gd = tq.tq_build_dictionary_device(dev, top_k=top_k)
    assert gd.K == od.K == hd.K
    assert np.array_equal(gd.entries, od.entries) and np.array_equal(gd.entries, hd.entries)
    assert np.array_equal(gd.counts, hd.counts)


# ------------------------------------------------------------------ device-side encoder
@pytest.mark.parametrize("rows,cols,spread,top_k", [(37, 516, 3, 300), (300, 3072, 6, 65535), (17, 8192, 4, 65535), (5, 4, 2, 10),
                                                    (64, 2048, 20, 65535), (48, 1280, 3, 0)])
def test_upload_device_builds_the_same_image_as_the_host(tq, rows, cols, spread, top_k):
    """tq_upload_device (levels on the GPU -> TILES image on the GPU) against tq_tiles_image_host
    fed with the oracle's stream: tokens, tile index, raw words, scales and zero points byte for
    byte; then the same y from both matrices."""
    rng = np.random.default_rng(rows + cols)
    q = np.clip(np.rint(rng.standard_t(5, size=(rows, cols)) * spread), -127, 127).astype(np.int8)
    s = (rng.random(rows) + 0.5).astype(np.float32)
    z = rng.integers(0, 5, rows).astype(np.float32)
    d, (stream,) = _oracle_pack([q], top_k=top_k)
    hd = tq.tq_dict_from_entries(d.entries)
    dd = tq.tq_dict_upload(hd)
    img, offs, steps, row_blocks = tq.tq_tiles_image_host(hd, stream, rows, cols, s, z)
    md = tq.tq_upload_device(dd, torch.from_numpy(q).cuda(), torch.from_numpy(s).cuda(), torch.from_numpy(z).cuda())
    got = md.buf.cpu().numpy()
    n_tiles = steps * row_blocks
    n_raw = int(img[offs["tile_raw"]:].view(np.uint32)[n_tiles])
    assert md.info.n_raw_words == n_raw and md.info.device_bytes == img.size
    assert md.info.n_hits + md.info.n_miss == rows * cols // 4 and md.info.stream_bytes == stream.nbytes
    for name, length in (("scale", 4 * row_blocks * 16), ("zero", 4 * row_blocks * 16), ("tile_raw", 4 * (n_tiles + 9)),
                         ("tokens", 1024 * n_tiles), ("raw", 4 * n_raw)):
        a, b = offs[name], offs[name] + length
        assert np.array_equal(got[a:b], img[a:b]), name
    mh = tq.tq_upload(dd, stream, rows, cols, s, z, layout=tq.TQ_LAYOUT_TILES)
    x = synth.activations(3, cols, 77).cuda()
    assert torch.equal(tq.tq_fused_gemv(md, x), tq.tq_fused_gemv(mh, x))
    assert np.array_equal(tq.tq_decompress(md).cpu().numpy(), q.view(np.uint8))
    assert tq.tq_device_status(md) == 0


# ------------------------------------------------------------------ stack: one persistent launch
@pytest.mark.parametrize("B", [1, 2, 3, 8, 11])
def test_stack_matches_oracle_and_single_calls(tq, B):
    """Several matrices of different shapes behind one table, one launch.  The integer sums make
    the result independent of how row blocks and columns are split among CTAs and warps, so the
    stack must reproduce the single-matrix calls bit for bit, and both must match the oracle."""
    shapes = [(300, 1024), (17, 8192), (1024, 3072), (16, 128), (530, 2052), (2048, 512)]
    rng = np.random.default_rng(100 + B)
    qs = [np.clip(np.rint(rng.standard_t(5, size=s) * 4), -127, 127).astype(np.int8) for s in shapes]
    ss = [(rng.random(r) + 0.5).astype(np.float32) for r, _ in shapes]
    d, streams = _oracle_pack(qs)
    dd = tq.tq_dict_upload(tq.tq_dict_from_entries(d.entries))
    mats = [tq.tq_upload(dd, st, r, c, s, layout=tq.TQ_LAYOUT_TILES) for st, (r, c), s in zip(streams, shapes, ss)]
    xs = [synth.activations(B, c, 300 + i).cuda() for i, (_, c) in enumerate(shapes)]
    ys = [torch.full((B, r), float("nan"), dtype=torch.float32, device="cuda") for r, _ in shapes]
    stack = tq.tq_stack_create(mats, xs, ys)
    # one vector: the kernel whose warps multiply on the spot; more: digit planes + one pass of the tcgen05 kernel
    # (two vectors do not fit beside the table for the 8192-column matrix)
    assert stack.launches == (1 if B == 1 else 2)
    for _ in range(2):  # a second launch reuses everything the first left behind
        for y in ys:
            y.fill_(float("nan"))
        tq.tq_fused_gemv_stack(stack)
        torch.cuda.synchronize()
        for m, q, s, x, y in zip(mats, qs, ss, xs, ys):
            single = tq.tq_fused_gemv(m, x)
            assert torch.equal(single, y)
            yref = oracle.layer_forward(q, s, x.cpu().double().numpy())
            assert _rel_err(y.cpu().numpy().astype(np.float64), yref) <= TIGHT
            assert tq.tq_device_status(m) == 0


@pytest.mark.parametrize("B", [1, 2])
@pytest.mark.parametrize("n_mats,max_rows", [(3, 40), (60, 200), (400, 48)])
def test_stack_of_many_small_matrices(tq, B, n_mats, max_rows):
    """Few small matrices leave most CTAs without a segment (they are not launched); hundreds of them
    give every CTA several segments of different matrices, each fetched as one record.  Unsigned levels
    with zero points, so the per-warp sums of x are used too.  Results: bit-equal to single calls, and
    within the tolerance of the oracle."""
    rng = np.random.default_rng(7000 + 10 * n_mats + B)
    shapes = [(int(rng.integers(1, max_rows + 1)), 4 * int(rng.integers(1, 300))) for _ in range(n_mats)]
    qs = [rng.integers(100, 140, size=s).astype(np.uint8) for s in shapes]
    ss = [(rng.random(r) + 0.5).astype(np.float32) for r, _ in shapes]
    zs = [rng.integers(110, 130, size=r).astype(np.float32) for r, _ in shapes]
    d, streams = _oracle_pack(qs, top_k=3000)
    dd = tq.tq_dict_upload(tq.tq_dict_from_entries(d.entries))
    mats = [tq.tq_upload(dd, st, r, c, s, z, levels_signed=False, layout=tq.TQ_LAYOUT_TILES)
            for st, (r, c), s, z in zip(streams, shapes, ss, zs)]
    xs = [synth.activations(B, c, 900 + i).cuda() for i, (_, c) in enumerate(shapes)]
    ys = [torch.full((B, r), float("nan"), dtype=torch.float32, device="cuda") for r, _ in shapes]
    stack = tq.tq_stack_create(mats, xs, ys)
    assert stack.launches == 1
    for _ in range(2):
        for y in ys:
            y.fill_(float("nan"))
        tq.tq_fused_gemv_stack(stack)
        torch.cuda.synchronize()
        for m, q, s, z, x, y in zip(mats, qs, ss, zs, xs, ys):
            assert torch.equal(tq.tq_fused_gemv(m, x), y)
            yref = oracle.layer_forward(q, s, x.cpu().double().numpy(), zero=z)
            assert _rel_err(y.cpu().numpy().astype(np.float64), yref) <= TIGHT
            assert tq.tq_device_status(m) == 0


@pytest.mark.parametrize("B", [1, 2, 5])
def test_stack_with_short_and_long_rows(tq, B):
    """Rows too long for a whole row of activation digits in shared memory (more than 8448 columns)
    take the tcgen05 kernel, whose B operand is staged step by step; a one-vector stack that mixes both
    kinds launches the narrow kernel for the short rows and the tcgen05 pair for the long ones."""
    shapes = [(200, 1024), (40, 12288), (600, 3072), (33, 28672), (64, 8192)]
    rng = np.random.default_rng(200 + B)
    qs = [np.clip(np.rint(rng.standard_t(5, size=s) * 4), -127, 127).astype(np.int8) for s in shapes]
    ss = [(rng.random(r) + 0.5).astype(np.float32) for r, _ in shapes]
    d, streams = _oracle_pack(qs, top_k=5000)
    dd = tq.tq_dict_upload(tq.tq_dict_from_entries(d.entries))
    mats = [tq.tq_upload(dd, st, r, c, s, layout=tq.TQ_LAYOUT_TILES) for st, (r, c), s in zip(streams, shapes, ss)]
    xs = [synth.activations(B, c, 400 + i).cuda() for i, (_, c) in enumerate(shapes)]
    ys = [torch.full((B, r), float("nan"), dtype=torch.float32, device="cuda") for r, _ in shapes]
    stack = tq.tq_stack_create(mats, xs, ys)
    # two vectors do not fit beside the table for 8192-column rows, so they and wider batches go through the
    # tcgen05 kernel for all matrices (digit planes + one pass)
    assert stack.launches == (3 if B == 1 else 2)
    tq.tq_fused_gemv_stack(stack)
    torch.cuda.synchronize()
    for m, q, s, x, y in zip(mats, qs, ss, xs, ys):
        assert torch.equal(tq.tq_fused_gemv(m, x), y)
        assert _rel_err(y.cpu().numpy().astype(np.float64), oracle.layer_forward(q, s, x.cpu().double().numpy())) <= TIGHT
        assert tq.tq_device_status(m) == 0


def test_decompress_stack_bit_exact(tq):
    """One persistent launch decompresses every matrix of a stack (ragged shapes, a table larger
    than the shared-memory limit so that some groups are stored raw); a stack may be made without
    operands for this purpose."""
    shapes = [(300, 1024), (17, 8192), (1000, 3072), (16, 128), (530, 2052), (1, 4)]
    rng = np.random.default_rng(41)
    qs = [rng.integers(-20, 21, size=s).astype(np.int8) for s in shapes]
    d, streams = _oracle_pack(qs)
    assert d.K > tq.TQ_TILES_TABLE_WORDS
    dd = tq.tq_dict_upload(tq.tq_dict_from_entries(d.entries))
    ones = [np.ones(r, dtype=np.float32) for r, _ in shapes]
    mats = [tq.tq_upload(dd, st, r, c, s, layout=tq.TQ_LAYOUT_TILES) for st, (r, c), s in zip(streams, shapes, ones)]
    assert sum(m.info.n_raw_words - m.info.n_miss for m in mats) > 0
    stack = tq.tq_stack_create(mats)
    outs = [torch.full((r * c,), 0x55, dtype=torch.uint8, device="cuda") for r, c in shapes]
    for _ in range(2):
        tq.tq_decompress_stack(stack, outs)
        torch.cuda.synchronize()
        for o, q, m, st in zip(outs, qs, mats, streams):
            assert np.array_equal(o.cpu().numpy().reshape(q.shape), d.decode(st).reshape(q.shape))
            assert np.array_equal(o.cpu().numpy().reshape(q.shape), q.view(np.uint8))
            assert tq.tq_device_status(m) == 0
    with pytest.raises(tq.TqError):
        tq.tq_fused_gemv_stack(stack)  # no operands were bound


def test_decode_bf16_stack_then_gemm(tq):
    """Phase 1 of the prefill product for all matrices of a stack in one launch, phase 2 per matrix."""
    shapes = [(300, 1024), (130, 8192), (1000, 3072), (16, 128)]
    rng = np.random.default_rng(43)
    qs = [np.clip(np.rint(rng.standard_t(5, size=s) * 5), -127, 127).astype(np.int8) for s in shapes]
    ss = [(rng.random(r) + 0.5).astype(np.float32) for r, _ in shapes]
    d, streams = _oracle_pack(qs)
    dd = tq.tq_dict_upload(tq.tq_dict_from_entries(d.entries))
    mats = [tq.tq_upload(dd, st, r, c, s, layout=tq.TQ_LAYOUT_TILES) for st, (r, c), s in zip(streams, shapes, ss)]
    stack = tq.tq_stack_create(mats)
    wss = [torch.full((tq.tq_gemm_workspace_size(m),), 0x7F, dtype=torch.uint8, device="cuda") for m in mats]
    tq.tq_decode_bf16_stack(stack, wss)
    M = 70
    for m, q, s, w, (r, c) in zip(mats, qs, ss, wss, shapes):
        X = synth.activations(M, c, 17)
        Y = tq.tq_gemm_bf16_ws(m, X.cuda(), w).cpu().numpy().astype(np.float64)
        assert _rel_err(Y, oracle.layer_forward(q, s, X.double().numpy())) <= GEMM_TIGHT
        # the workspace holds the levels themselves as bf16, in whole tiles
        rows_pad, pitch = -(-r // 16) * 16, -(-c // 128) * 128
        wb = w.view(torch.bfloat16)[: rows_pad * pitch].view(rows_pad, pitch)[:r, :c].float().cpu().numpy()
        assert np.array_equal(wb, q.astype(np.float32))
        assert tq.tq_device_status(m) == 0


def test_stack_rejects_mixed_tables_and_layouts(tq):
    rng = np.random.default_rng(9)
    q = rng.integers(-3, 4, size=(32, 256)).astype(np.int8)
    s = np.ones(32, dtype=np.float32)
    d, (stream,) = _oracle_pack([q])
    dd1 = tq.tq_dict_upload(tq.tq_dict_from_entries(d.entries))
    dd2 = tq.tq_dict_upload(tq.tq_dict_from_entries(d.entries))
    a = tq.tq_upload(dd1, stream, 32, 256, s, layout=tq.TQ_LAYOUT_TILES)
    b = tq.tq_upload(dd2, stream, 32, 256, s, layout=tq.TQ_LAYOUT_TILES)
    c = tq.tq_upload(dd1, stream, 32, 256, s, layout=tq.TQ_LAYOUT_PLANES)
    x = synth.activations(1, 256, 1).cuda()
    y = torch.empty((1, 32), dtype=torch.float32, device="cuda")
    for pair in ([a, b], [a, c]):
        with pytest.raises(tq.TqError) as e:
            tq.tq_stack_create(pair, [x, x], [y, y.clone()])
        assert e.value.status == tq.TQ_ERR_UNSUPPORTED_SHAPE


# ------------------------------------------------------------------ full size, as benchmarked
@pytest.fixture(scope="module")
def model3b(tq):
    """The whole LLaMA-3.2-3B linear stack (197 matrices, 3.2 G weights) built by the benchmark's own
    builder, with 32 activation vectors per matrix; smaller batches use the first vectors."""
    import bench

    shapes = synth.llama32_linear_shapes("3b")
    device = torch.device("cuda", 0)
    mats, xs, ys, hd, q_host, scales, stats, x_arena, y_arena, dd = bench.build_model(
        tq, shapes, 32, device, 0, None, layout=tq.TQ_LAYOUT_TILES)
    yield {"shapes": shapes, "device": device, "mats": mats, "xs": xs, "ys": ys, "hd": hd, "q_host": q_host,
           "scales": scales, "y_arena": y_arena}
    del mats, xs, ys, x_arena, y_arena
    torch.cuda.empty_cache()


@pytest.mark.parametrize("B", [1, 8, 32])
def test_full_3b_stack_as_benchmarked_on_sampled_rows(tq, model3b, B):
    """The launch configuration the benchmark times (one tq_fused_gemv_stack call over all 197
    matrices) at 1, 8 and 32 vectors.  The oracle regenerates sampled rows, quantizes them itself and
    computes their outputs one by one; decoded levels of those rows must match bit for bit."""
    shapes, device, mats, q_host, scales = (model3b[k] for k in ("shapes", "device", "mats", "q_host", "scales"))
    xs = [x[:B] for x in model3b["xs"]]
    ys = [torch.full((B, r), float("nan"), dtype=torch.float32, device=device) for _, r, _ in shapes]
    stack = tq.tq_stack_create(mats, xs, ys)
    tq.tq_fused_gemv_stack(stack)
    torch.cuda.synchronize()
    assert not any(bool(torch.isnan(y).any()) for y in ys)
    rng = np.random.default_rng(2025 + B)
    picks = [0, 1, 2, 3, 4, 5, 6, 97, 100, 103, 190, 195, 196]  # every kind of layer, first/middle/last, lm_head
    for i in picks:
        name, rows, cols = shapes[i]
        sample = np.sort(rng.choice(rows, 24, replace=False))
        sample[0], sample[-1] = 0, rows - 1
        w = synth.weight(rows, cols, synth.matrix_seed(i), device=device)[torch.from_numpy(sample).to(device)].cpu().numpy()
        qo, so = oracle.quantize_rows(w)
        assert np.array_equal(qo, q_host[i][sample]) and np.array_equal(so, scales[i][sample])
        yref = oracle.layer_forward(qo, so, xs[i].cpu().double().numpy())
        y = ys[i][:, torch.from_numpy(sample).to(device)].cpu().numpy().astype(np.float64)
        err = np.max(np.abs(y - yref), axis=1) / np.max(np.abs(yref), axis=1)
        assert float(err.max()) <= TIGHT, (name, err)
        assert tq.tq_device_status(mats[i]) == 0


def test_full_3b_table_and_decompress_stack(tq, model3b):
    """The table was built with the counting on the GPU: it must be the host builder's table.  Then
    tq_decompress_stack of the whole set (3.2 GB of levels, one persistent launch), every matrix
    compared with the levels that were encoded."""
    mats, q_host, hd, device = (model3b[k] for k in ("mats", "q_host", "hd", "device"))
    assert np.array_equal(hd.entries, tq.tq_build_dictionary(q_host).entries)
    outs = [torch.full((m.info.rows * m.info.cols,), 0x55, dtype=torch.uint8, device=device) for m in mats]
    tq.tq_decompress_stack(tq.tq_stack_create(mats), outs)
    torch.cuda.synchronize()
    for o, q, m in zip(outs, q_host, mats):
        assert torch.equal(o.view(torch.int8), torch.from_numpy(q).to(device).view(-1))
        assert tq.tq_device_status(m) == 0
    # and the single-matrix call on one decoder matrix and on the output head
    for i in (6, 196):
        got = tq.tq_decompress(mats[i])
        assert np.array_equal(got.cpu().numpy().view(np.int8), q_host[i])
        del got


def test_full_3b_prefill_group_at_2048_tokens(tq, model3b):
    """The prefill leg as the benchmark launches it: 14 decoder layers (98 matrices) decoded to bf16 by
    one launch, then all their products at M = 2048 tokens by one tq_gemm_plan_run launch; sampled
    (token, row) outputs against the oracle."""
    shapes, device, mats, q_host, scales = (model3b[k] for k in ("shapes", "device", "mats", "q_host", "scales"))
    M, group = 2048, list(range(98))
    gm = [mats[i] for i in group]
    Xs = {c: synth.activations(M, c, 99, device=device) for c in sorted({m.info.cols for m in gm})}
    wss = [torch.empty(tq.tq_gemm_workspace_size(m), dtype=torch.uint8, device=device) for m in gm]
    plan = tq.tq_gemm_plan_create(gm, [Xs[m.info.cols] for m in gm], wss)
    tq.tq_decode_bf16_stack(tq.tq_stack_create(gm), wss)
    tq.tq_gemm_plan_run(plan)
    torch.cuda.synchronize()
    assert tq.tq_gemm_plan_status(plan) == 0
    rng = np.random.default_rng(77)
    for k in (0, 1, 3, 5, 6, 49, 52, 91, 97):
        i = group[k]
        name, rows, cols = shapes[i]
        rsel = np.sort(rng.choice(rows, 16, replace=False))
        tsel = np.sort(rng.choice(M, 12, replace=False))
        tsel[0], tsel[-1] = 0, M - 1
        yref = oracle.layer_forward(q_host[i][rsel], scales[i][rsel], Xs[cols][torch.from_numpy(tsel).to(device)].cpu().double().numpy())
        y = plan.Ys[k][torch.from_numpy(tsel).to(device)][:, torch.from_numpy(rsel).to(device)].cpu().numpy().astype(np.float64)
        assert _rel_err(y, yref) <= GEMM_TIGHT, name
        assert tq.tq_device_status(mats[i]) == 0


# ------------------------------------------------------------------ row shards (the multi-GPU split, on one GPU)
@pytest.mark.parametrize("B", [1, 8])
@pytest.mark.parametrize("world", [2, 3])
def test_row_shards_reproduce_the_unsharded_product(tq, B, world):
    """The split a multi-GPU run makes (output rows in whole blocks of 16 per rank, same table), run
    here one shard after the other on one GPU: shard outputs concatenated must equal the unsharded
    call bit for bit (the sums are exact integers, so no split can change them), decoded levels of the
    shards must be the matrix's rows, and the one-arena-per-rank layout must reassemble the stack."""
    from paper_2509_22951_b200 import sharding

    shapes = [("a", 1000, 3072), ("b", 300, 1024), ("c", 16, 128), ("d", 130, 8192)]
    rng = np.random.default_rng(500 + B + world)
    qs = [np.clip(np.rint(rng.standard_t(5, size=(r, c)) * 5), -127, 127).astype(np.int8) for _, r, c in shapes]
    ss = [(rng.random(r) + 0.5).astype(np.float32) for _, r, _ in shapes]
    d, _ = _oracle_pack(qs)
    dd = tq.tq_dict_upload(tq.tq_dict_from_entries(d.entries))
    qd = [torch.from_numpy(q).cuda() for q in qs]
    sd = [torch.from_numpy(s).cuda() for s in ss]
    xs = [synth.activations(B, c, 600 + i).cuda() for i, (_, _, c) in enumerate(shapes)]
    whole = [tq.tq_upload_device(dd, q, s) for q, s in zip(qd, sd)]
    y_whole = [tq.tq_fused_gemv(m, x) for m, x in zip(whole, xs)]
    so = sharding.ShardedOutputs(shapes, B, world)
    arenas = []
    for rank in range(world):
        mats = sharding.upload_row_shards(tq, dd, qd, sd, rank, world)
        arena = torch.full((so.arena_len,), float("nan"), dtype=torch.float32, device="cuda")
        views = so.local_views(arena, rank)
        have = [i for i, m in enumerate(mats) if m is not None]
        if have:
            tq.tq_fused_gemv_stack(tq.tq_stack_create([mats[i] for i in have], [xs[i] for i in have], [views[i] for i in have]))
        torch.cuda.synchronize()
        for i in have:
            r0, r1 = so.ranges[rank][i]
            assert np.array_equal(tq.tq_decompress(mats[i]).cpu().numpy().view(np.int8), qs[i][r0:r1])
            assert tq.tq_device_status(mats[i]) == 0
        arenas.append(arena)
    gathered = torch.cat(arenas)  # what one all-gather leaves on every rank
    for i, (_, rows, cols) in enumerate(shapes):
        y = so.full_output(gathered, i)
        assert torch.equal(y, y_whole[i])
        yref = oracle.layer_forward(qs[i], ss[i], xs[i].cpu().double().numpy())
        assert _rel_err(y.cpu().numpy().astype(np.float64), yref) <= TIGHT


def test_row_shard_rejects_unaligned_start(tq):
    q = torch.zeros((40, 12), dtype=torch.int8, device="cuda")  # 12-byte rows: row 1 starts on byte 12
    s = torch.ones(40, dtype=torch.float32, device="cuda")
    dd = tq.tq_dict_upload(tq.tq_dict_from_entries(np.zeros((1, 4), dtype=np.uint8)))
    with pytest.raises(tq.TqError) as e:
        tq.tq_upload_device_rows(dd, q, 1, 17, s)
    assert e.value.status == tq.TQ_ERR_INVALID_ARG
    m = tq.tq_upload_device_rows(dd, q, 4, 20, s)  # row 4 starts on byte 48
    assert m.info.rows == 16 and m.info.cols == 12


# ------------------------------------------------------------------ bounded waits
def test_expired_wait_is_reported_and_the_context_survives(tq):
    """The waits inside the kernels are bounded.  With the library's test hook on, the one-vector kernel
    expects a chunk of the table that is never copied: the waits run out (about 2 s), the kernel ends by
    itself, the status word says so, and the next, ordinary call on the same matrix is correct."""
    rng = np.random.default_rng(321)
    q = np.clip(np.rint(rng.standard_t(5, size=(64, 1024)) * 4), -127, 127).astype(np.int8)
    s = (rng.random(64) + 0.5).astype(np.float32)
    d, (stream,) = _oracle_pack([q])
    m = _upload_from_oracle(tq, d, stream, 64, 1024, s, layout=tq.TQ_LAYOUT_TILES)
    x = synth.activations(1, 1024, 3)
    yref = oracle.layer_forward(q, s, x.double().numpy())
    tq.tq_test_withhold_table_chunk(True)
    try:
        tq.tq_fused_gemv(m, x.cuda())
        torch.cuda.synchronize()
    finally:
        tq.tq_test_withhold_table_chunk(False)
    assert tq.tq_device_status(m) == tq.TQ_STATUS_WAIT_EXPIRED
    y = tq.tq_fused_gemv(m, x.cuda()).cpu().numpy().astype(np.float64)
    assert _rel_err(y, yref) <= TIGHT
    assert tq.tq_device_status(m) == 0
