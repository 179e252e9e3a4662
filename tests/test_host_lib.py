"""Host half of libtq against the oracle: quantizers, table, encoder, stream validation.  No GPU."""
import ctypes
import os
import re

import numpy as np
import pytest

from inputs import synth
from oracle import oracle
from paper_2509_22951_b200 import binding as tq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "tq.h")).read()
    declared = set(re.findall(r"\b(tq_[a-z0-9_]+)\s*\(", hdr))
    assert declared, "no declarations found"
    lib = ctypes.CDLL(str(tq._build.LIB))
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} declared in tq.h but not exported"
    assert declared == set(tq.EXPORTS)


def test_quantize_rows_matches_oracle_bit_exact():
    w = synth.weight(96, 512, synth.matrix_seed(3)).numpy()
    w[5] = 0
    q, s = tq.tq_quantize_rows(w)
    qo, so = oracle.quantize_rows(w)
    assert np.array_equal(q, qo) and np.array_equal(s, so)


def test_quantize_tensor_matches_oracle_bit_exact():
    x = synth.weight(64, 256, synth.matrix_seed(4)).numpy()
    q, s, z = tq.tq_quantize_tensor(x)
    qo, so, zo = oracle.quantize_paper(x)
    assert np.array_equal(q, qo) and s == so and z == zo
    with pytest.raises(tq.TqError):
        tq.tq_quantize_tensor(np.zeros(16, dtype=np.float32))


@pytest.mark.parametrize("bits", [1, 2, 4, 6, 8])
def test_quantize_tensor_bits_matches_oracle_bit_exact(bits):
    x = synth.weight(48, 320, synth.matrix_seed(5)).numpy()
    q, s, z = tq.tq_quantize_tensor_bits(x, bits)
    qo, so, zo = oracle.quantize_paper(x, bits=bits)
    assert np.array_equal(q, qo) and s == so and z == zo and q.max() == 2 ** bits - 1
    for bad in (0, 9):
        with pytest.raises(tq.TqError):
            tq.tq_quantize_tensor_bits(x, bad)


def _check_same(mats, top_k):
    d = tq.tq_build_dictionary(mats, top_k)
    o = oracle.Dictionary.build(mats, top_k)
    assert d.K == o.K
    assert np.array_equal(d.entries, o.entries)
    assert np.array_equal(d.counts, o.counts)
    for m in mats:
        s, h, mi = tq.tq_encode(d, m)
        so, ho, mo = o.encode(m)
        assert (h, mi) == (ho, mo) and np.array_equal(s, so)
        assert np.array_equal(o.decode(s), np.ascontiguousarray(m).view(np.uint8).ravel())
    return d, o


@pytest.mark.parametrize("seed", range(8))
@pytest.mark.parametrize("threads", [1, 3])
def test_dictionary_and_stream_identical_small_alphabets(seed, threads):
    tq.tq_set_num_threads(threads)
    try:
        rng = np.random.default_rng(seed)
        a = int(rng.integers(1, 9))
        mats = [rng.integers(0, a + 1, size=int(rng.integers(0, 5000))).astype(np.uint8)
                for _ in range(int(rng.integers(1, 5)))]
        for top_k in (65535, 50, 3, 0):
            _check_same(mats, top_k)
    finally:
        tq.tq_set_num_threads(0)


def test_dictionary_many_ties_at_the_cut():
    # ~all windows distinct: the cut falls inside a huge class of count-1 windows, so the table is
    # the first 65534 windows in visiting order
    rng = np.random.default_rng(1)
    data = rng.integers(0, 256, size=300_000).astype(np.uint8)
    d, o = _check_same([data], 65535)
    assert d.K == 65534


def test_dictionary_tie_walk_path(monkeypatch):
    # force the in-order walk that picks first-seen windows out of a large tied class
    monkeypatch.setenv("TQ_TIE_LIMIT", "10")
    rng = np.random.default_rng(2)
    mats = [rng.integers(0, 4, size=3000).astype(np.uint8), rng.integers(0, 7, size=2000).astype(np.uint8)]
    for top_k in (65535, 400, 120, 30, 5, 1):
        _check_same(mats, top_k)


def test_dictionary_multithreaded_large_matches_oracle():
    # config-0 sized layer, quantized weights, several threads and buckets
    w = synth.weight(1024, 2048, synth.matrix_seed(0)).numpy()
    q, s = oracle.quantize_rows(w)
    w2 = synth.weight(512, 2048, synth.matrix_seed(1)).numpy()
    q2, s2 = oracle.quantize_rows(w2)
    tq.tq_set_num_threads(4)
    try:
        _check_same([q, q2], 65535)
    finally:
        tq.tq_set_num_threads(0)


def test_encode_tails_and_buffer_check():
    d = tq.tq_dict_from_entries(np.array([[1, 2, 3, 4]], dtype=np.uint8))
    o = oracle.Dictionary.from_entries(np.array([[1, 2, 3, 4]], dtype=np.uint8))
    for n in range(0, 14):
        data = np.array(([1, 2, 3, 4, 9, 8, 7, 6] * 2)[:n], dtype=np.uint8)
        s, h, m = tq.tq_encode(d, data)
        so, _, _ = o.encode(data)
        assert np.array_equal(s, so)
    data = np.arange(8, dtype=np.uint8)
    n = ctypes.c_uint64()
    out = np.zeros(3, dtype=np.uint16)
    rc = tq._lib.tq_encode(d._h, tq._np_ptr(data, ctypes.c_uint8), 8, tq._np_ptr(out, ctypes.c_uint16), 3,
                           ctypes.byref(n), None, None)
    assert rc == tq.TQ_ERR_BUFFER_TOO_SMALL and n.value == 10


# ------------------------------------------------------------------ stream validation (host part of tq_upload)
def _valid_stream(rows=6, cols=16, seed=0):
    rng = np.random.default_rng(seed)
    q = rng.integers(0, 3, size=(rows, cols)).astype(np.uint8)
    o = oracle.Dictionary.build([q], top_k=5)
    s, h, m = o.encode(q)
    assert h > 0 and m > 0
    return s, rows, cols


@pytest.mark.parametrize("layout", [0, 1], ids=["stream", "planes"])
def test_upload_size_accepts_valid_and_rejects_corrupt(layout):
    s, rows, cols = _valid_stream()
    assert tq.tq_upload_size(s, rows, cols, layout) > 0

    def bad(stream, r=rows, c=cols):
        with pytest.raises(tq.TqError) as e:
            tq.tq_upload_size(stream, r, c, layout)
        return e.value.status

    assert bad(s[:-1]) == tq.TQ_ERR_CORRUPT_STREAM               # truncated
    assert bad(np.append(s, 1).astype(np.uint16)) == tq.TQ_ERR_CORRUPT_STREAM  # one group too many
    esc = int(np.flatnonzero(s == 0xFFFF)[0])
    t = s.copy(); t[esc + 2] = 300                                 # raw slot > 255
    assert bad(t) == tq.TQ_ERR_CORRUPT_STREAM
    t = s.copy(); t[esc + 1] = 0xFFFF                              # marker inside raw run
    assert bad(t) == tq.TQ_ERR_CORRUPT_STREAM
    code = int(np.flatnonzero((s != 0xFFFF) & (s > 0) & (np.arange(s.size) > 4))[0])
    t = s.copy()
    if not any(t[max(0, code - 4):code] == 0xFFFF):
        t[code] = 0                                                # code 0 is never assigned
        assert bad(t) == tq.TQ_ERR_CORRUPT_STREAM
    assert bad(s, rows, cols + 2) == tq.TQ_ERR_UNSUPPORTED_SHAPE   # cols % 4 != 0
    assert bad(s, rows + 1, cols) == tq.TQ_ERR_CORRUPT_STREAM      # wrong shape for this stream
    t = np.concatenate([s[:-5], [0xFFFF, 1, 2, 3]]).astype(np.uint16) if s[-5] == 0xFFFF else None
    if t is not None:
        assert bad(t) == tq.TQ_ERR_CORRUPT_STREAM                  # marker with < 4 slots after it


def test_row_partition_helper_two_ranks_gloo():
    """Row sharding for several GPUs is a plain split of the rows: check with 2 gloo ranks that the
    shards tile the matrix in whole blocks of 16 rows, that concatenating per-rank oracle outputs
    gives the full output, and that the one-collective-per-stack arena layout reassembles every
    matrix of a stack."""
    import torch.multiprocessing as mp
    mp.spawn(_rank_main, args=(2,), nprocs=2, join=True)


def _rank_main(rank, world):
    import torch
    import torch.distributed as dist
    from paper_2509_22951_b200 import sharding
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29531")
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rng = np.random.default_rng(7)
        shapes = [("a", 37, 16), ("b", 64, 8), ("c", 5, 12), ("d", 100, 4)]
        B = 3
        qs = [rng.integers(-127, 128, size=(r, c)).astype(np.int8) for _, r, c in shapes]
        ss = [(rng.random(r) + 0.5).astype(np.float32) for _, r, _ in shapes]
        xs = [rng.standard_normal((B, c)) for _, _, c in shapes]
        # single matrix
        rows = shapes[0][1]
        r0, r1 = sharding.row_range(rows, rank, world)
        y_local = torch.from_numpy(oracle.layer_forward(qs[0][r0:r1], ss[0][r0:r1], xs[0]))
        parts = sharding.all_gather_rows(y_local, rows, rank, world)
        assert torch.equal(parts, torch.from_numpy(oracle.layer_forward(qs[0], ss[0], xs[0])))
        # shards tile [0, rows) in whole blocks of 16 rows; 5 rows over 2 ranks leave one rank empty
        for _, rows, _ in shapes:
            cover = [sharding.row_range(rows, r, world) for r in range(world)]
            assert cover[0][0] == 0 and cover[-1][1] == rows and all(a[1] == b[0] for a, b in zip(cover, cover[1:]))
            assert all(a % 16 == 0 for a, _ in cover)
        assert sharding.row_range(5, 0, 2) == (0, 0) and sharding.row_range(5, 1, 2) == (0, 5)
        # a stack: every rank writes its slices into its arena, one all-gather, every matrix reassembled
        so = sharding.ShardedOutputs(shapes, B, world)
        arena = torch.zeros(so.arena_len, dtype=torch.float64)
        for i, view in enumerate(so.local_views(arena, rank)):
            a, b = so.ranges[rank][i]
            if b > a:
                view.copy_(torch.from_numpy(oracle.layer_forward(qs[i][a:b], ss[i][a:b], xs[i])))
        gathered = so.all_gather(arena)
        for i in range(len(shapes)):
            assert torch.equal(so.full_output(gathered, i), torch.from_numpy(oracle.layer_forward(qs[i], ss[i], xs[i])))
    finally:
        dist.destroy_process_group()


def _decode_tiles_image(img, offs, steps, row_blocks, rows, cols, entries):
    """Walks a TQ_LAYOUT_TILES image the way the layout is documented and returns the levels."""
    n_tiles = steps * row_blocks
    tile_raw = img[offs["tile_raw"]:offs["tile_raw"] + 4 * (n_tiles + 1)].view(np.uint32)
    tokens = img[offs["tokens"]:offs["tokens"] + 1024 * n_tiles].view(np.uint16).reshape(n_tiles, 2, 32, 8)
    raw = img[offs["raw"]:].view(np.uint32)
    table = np.zeros((65536, 4), dtype=np.uint8)
    table[1:1 + len(entries)] = entries
    out = np.zeros((row_blocks * 16, steps * 128), dtype=np.uint8)
    for tile in range(n_tiles):
        rb, s = divmod(tile, steps)
        first, end = int(tile_raw[tile]), int(tile_raw[tile + 1])
        used = set()
        for lane in range(32):
            g, t = lane >> 2, lane & 3
            for h in range(2):
                for i in range(8):
                    tk = int(tokens[tile, h, lane, i])
                    if tk >= 0xFC00:  # miss: the token is the ring slot of its raw word
                        p = first + ((tk - first) & 1023)
                        assert first <= p < end and p not in used
                        used.add(p)
                        w = np.array([raw[p]], dtype=np.uint32).view(np.uint8)
                    else:
                        assert tk < tq.TQ_TILES_TABLE_WORDS
                        w = table[tk]
                    c0 = 4 * (32 * s + 8 * t + i)
                    out[rb * 16 + g + 8 * h, c0:c0 + 4] = w
        assert len(used) == end - first
    assert not out[rows:].any() and not out[:, cols:].any()  # padding decodes to zeros
    return out[:rows, :cols]


@pytest.mark.parametrize("rows,cols,top_k", [(16, 128, 50), (37, 516, 300), (5, 4, 10), (48, 1280, 0), (33, 260, 65535)])
def test_tiles_image_decodes_to_the_original_levels(rows, cols, top_k):
    rng = np.random.default_rng(rows * 7 + cols)
    q = np.clip(np.rint(rng.standard_t(5, size=(rows, cols)) * 3), -127, 127).astype(np.int8)
    d = oracle.Dictionary.build([q], top_k=top_k)
    stream = d.encode(q)[0]
    s = (rng.random(rows) + 0.5).astype(np.float32)
    z = rng.integers(0, 9, rows).astype(np.float32)
    hd = tq.tq_dict_from_entries(d.entries)
    img, offs, steps, row_blocks = tq.tq_tiles_image_host(hd, stream, rows, cols, s, z)
    assert steps == -(-cols // 128) and row_blocks == -(-rows // 16)
    got = _decode_tiles_image(img, offs, steps, row_blocks, rows, cols, d.entries)
    assert np.array_equal(got, q.view(np.uint8))
    assert np.array_equal(img[offs["scale"]:offs["scale"] + 4 * rows].view(np.float32), s)
    assert np.array_equal(img[offs["zero"]:offs["zero"] + 4 * rows].view(np.float32), z)
    n_miss = int(np.count_nonzero(stream == 0xFFFF))
    assert int(img[offs["tile_raw"]:].view(np.uint32)[steps * row_blocks]) == n_miss


def test_tiles_image_stores_codes_beyond_the_shared_memory_table_as_raw_words():
    # a table with 65534 entries: groups coded at or beyond TQ_TILES_TABLE_WORDS become raw words
    rng = np.random.default_rng(77)
    q = rng.integers(-20, 21, size=(64, 2048)).astype(np.int8)
    d = oracle.Dictionary.build([q])
    assert d.K == 65534
    stream = d.encode(q)[0]
    far = int(np.count_nonzero((stream >= tq.TQ_TILES_TABLE_WORDS) & (stream != 0xFFFF) & _code_slots(stream)))
    assert far > 0
    s = np.ones(64, dtype=np.float32)
    hd = tq.tq_dict_from_entries(d.entries)
    img, offs, steps, row_blocks = tq.tq_tiles_image_host(hd, stream, 64, 2048, s)
    got = _decode_tiles_image(img, offs, steps, row_blocks, 64, 2048, d.entries)
    assert np.array_equal(got, q.view(np.uint8))
    n_miss = int(np.count_nonzero(stream == 0xFFFF))
    assert int(img[offs["tile_raw"]:].view(np.uint32)[steps * row_blocks]) == n_miss + far


def _code_slots(stream):
    """True at the slots of a token stream that hold a code or a marker (not a raw value)."""
    esc = np.flatnonzero(stream == 0xFFFF)
    mask = np.ones(stream.size, dtype=bool)
    for k in range(1, 5):
        mask[esc + k] = False
    return mask


@pytest.mark.parametrize("n_ctas", [1, 7, 148])
def test_stack_plan_covers_every_row_block_once_and_balances_cost(n_ctas):
    """The persistent kernels trust this split: every row block of every matrix must fall in exactly
    one segment, segments must come in matrix order, and the shares must cost about the same."""
    rng = np.random.default_rng(n_ctas)
    shapes = [(3072, 3072), (1024, 3072), (1024, 3072), (3072, 3072), (8192, 3072), (8192, 3072), (3072, 8192)] * 4
    shapes += [(128256, 3072), (17, 4), (16, 128)]
    steps = [-(-c // 128) for _, c in shapes]
    row_blocks = [-(-r // 16) for r, _ in shapes]
    rb_raw = []
    for s_, nrb in zip(steps, row_blocks):  # raw words per row block: about 55 % of the 512 groups of a tile
        per = rng.binomial(512 * s_, 0.55, size=nrb).astype(np.uint64)
        rb_raw.append(np.concatenate([[0], np.cumsum(per)]).astype(np.uint32))
    segs, cta_seg = tq.tq_stack_plan_host(steps, row_blocks, rb_raw, n_ctas)
    assert len(cta_seg) == n_ctas + 1 and cta_seg[0] == 0 and cta_seg[-1] == len(segs)
    assert all(a <= b for a, b in zip(cta_seg, cta_seg[1:]))
    nxt = [0] * len(shapes)
    order = []
    for m, b, e in segs:
        assert b == nxt[m] and b < e <= row_blocks[m]
        nxt[m] = e
        order.append(m)
    assert nxt == row_blocks and order == sorted(order)

    def cost(m, b, e):
        return (e - b) * steps[m] * 1024 + 4 * (int(rb_raw[m][e]) - int(rb_raw[m][b]))

    share = [sum(cost(*segs[i]) for i in range(cta_seg[c], cta_seg[c + 1])) for c in range(n_ctas)]
    total = sum(share)
    assert total == sum(cost(m, 0, row_blocks[m]) for m in range(len(shapes)))
    if n_ctas > 1:
        biggest_block = max(cost(m, 0, 1) for m in range(len(shapes))) * 2
        charge = 384 * 1024  # what the split charges per segment start, in bytes of stream
        assert max(share) <= total / n_ctas + biggest_block + (len(shapes) + n_ctas) * charge / n_ctas + charge * 3
