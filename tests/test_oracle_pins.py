"""Pins for the CPU oracle: everything here checks oracle/ against something other
than itself -- hand-worked fixtures, closed forms, invariants, brute force on tiny
inputs, and library routines.  No GPU, no CUDA library.
"""
import json
import os

import numpy as np
import pytest

from oracle import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")
ESC = 0xFFFF


def _load(name):
    with open(os.path.join(GOLD, name)) as f:
        return json.load(f)["cases"]


# ----------------------------------------------------------------------------
# Hand-worked fixtures (Listings 1-4)
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("case", _load("handworked_streams.json"), ids=lambda c: c["cite"][:40])
def test_handworked_streams(case):
    L = case.get("seq", 4)
    d = oracle.Dictionary.from_entries(np.array(case["table"], dtype=np.uint8).reshape(-1, L), seq=L)
    data = np.array(case["bytes"], dtype=np.uint8)
    stream, hits, miss = d.encode(data)
    assert stream.dtype == np.uint16
    assert stream.tolist() == case["stream"]
    assert d.decode(np.array(case["stream"], dtype=np.uint16)).tolist() == case["bytes"]
    nb, r = divmod(len(case["bytes"]), L)
    assert hits + miss == nb
    assert len(case["stream"]) == hits + (1 + L) * miss + ((1 + r) if r else 0)


@pytest.mark.parametrize("case", _load("handworked_tables.json"), ids=lambda c: c["cite"][:40])
def test_handworked_tables(case):
    mats = [np.array(m, dtype=np.uint8) for m in case["mats"]]
    d = oracle.Dictionary.build(mats, top_k=case["top_k"], seq=case.get("seq", 4))
    assert d.entries.tolist() == case["entries"]
    assert d.counts.tolist() == case["counts"]


@pytest.mark.parametrize("case", _load("handworked_quantizer.json"), ids=lambda c: c["cite"][:40])
def test_handworked_quantizer(case):
    q, s, z = oracle.quantize_paper(np.array(case["x"], dtype=np.float32), bits=case.get("bits", 8))
    assert q.tolist() == case["q"]
    assert s == np.float32(case["scale_num"]) / np.float32(case["scale_den"])
    assert z == np.float32(case["zero"])


# ----------------------------------------------------------------------------
# Dictionary: brute force on tiny inputs (O(n^2) counting, different algorithm)
# ----------------------------------------------------------------------------
def _brute_table(mats, top_k, L=4):
    wins = []  # every window, in visiting order
    for m in mats:
        m = list(m)
        for i in range(len(m) - L + 1):
            wins.append(tuple(m[i:i + L]))
    ranked = []
    for i, w in enumerate(wins):
        first = min(j for j in range(len(wins)) if wins[j] == w)
        if first != i:
            continue
        cnt = sum(1 for v in wins if v == w)
        ranked.append((-cnt, first, w))
    ranked.sort()
    keep = min(top_k, 65534)
    return [list(w) for _, _, w in ranked[:keep]], [-c for c, _, _ in ranked[:keep]], len(ranked), len(wins)


@pytest.mark.parametrize("seed", range(12))
def test_dictionary_brute_force(seed):
    rng = np.random.default_rng(seed)
    n_mats = int(rng.integers(1, 4))
    alphabet = int(rng.integers(1, 4))  # tiny alphabets force repeats and ties
    mats = [rng.integers(0, alphabet + 1, size=int(rng.integers(0, 120))).astype(np.uint8)
            for _ in range(n_mats)]
    for top_k in (65535, 7, 1, 0):
        want_e, want_c, n_distinct, n_win = _brute_table(mats, top_k)
        d = oracle.Dictionary.build(mats, top_k=top_k)
        assert d.entries.tolist() == want_e
        assert d.counts.tolist() == want_c
        assert d.n_distinct == n_distinct
        assert d.n_windows == n_win == sum(max(0, len(m) - 3) for m in mats)
    # Listing 2's sequence_length at 2 and 8: same brute force, windows of that length
    for L in (2, 8):
        for top_k in (65535, 3):
            want_e, want_c, n_distinct, n_win = _brute_table(mats, top_k, L)
            d = oracle.Dictionary.build(mats, top_k=top_k, seq=L)
            assert d.entries.tolist() == want_e and d.counts.tolist() == want_c
            assert d.n_distinct == n_distinct
            assert d.n_windows == n_win == sum(max(0, len(m) - L + 1) for m in mats)


def test_dictionary_invariants_and_escape_collision():
    rng = np.random.default_rng(99)
    data = rng.integers(0, 256, size=400_000).astype(np.uint8)  # ~all windows distinct
    d = oracle.Dictionary.build([data], top_k=2 ** 16 - 1)
    # code 65535 is the escape marker, so at most 65534 entries are usable
    assert d.n_distinct > 65535 and d.K == 65534
    c = d.counts.astype(np.int64)
    assert np.all(c[:-1] >= c[1:])  # counts never increase with rank
    assert d.n_windows == data.size - 3
    e = d.entries
    assert len({tuple(r) for r in e.tolist()}) == d.K  # entries are distinct
    # full table on a small input: counts sum to the number of windows
    small = rng.integers(0, 3, size=5000).astype(np.uint8)
    ds = oracle.Dictionary.build([small])
    assert ds.K == ds.n_distinct and int(ds.counts.sum()) == small.size - 3


# ----------------------------------------------------------------------------
# Encoder / decoder: round trip, size identity, closed forms, structure
# ----------------------------------------------------------------------------
def _classify(stream):
    """Independent walk of a stream: returns (#codes, #escapes-with-4, tail_len)."""
    i, codes, esc, tail = 0, 0, 0, 0
    s = stream.tolist()
    while i < len(s):
        if s[i] == ESC:
            k = min(4, len(s) - i - 1)
            assert all(v <= 255 for v in s[i + 1:i + 1 + k])
            if k == 4:
                esc += 1
            else:
                tail = k
            i += 5
        else:
            codes += 1
            i += 1
    return codes, esc, tail


@pytest.mark.parametrize("n", [0, 1, 2, 3, 4, 5, 7, 8, 1023, 4096, 4097, 4098, 4099])
@pytest.mark.parametrize("alphabet,top_k", [(2, 65535), (5, 16), (256, 65535), (4, 0)])
def test_round_trip_and_size_identity(n, alphabet, top_k):
    rng = np.random.default_rng(n * 31 + alphabet)
    data = rng.integers(0, alphabet, size=n).astype(np.uint8)
    other = rng.integers(0, alphabet, size=257).astype(np.uint8)
    d = oracle.Dictionary.build([data, other], top_k=top_k)
    stream, hits, miss = d.encode(data)
    nb, r = divmod(n, 4)
    assert hits + miss == nb
    assert stream.size == hits + 5 * miss + ((1 + r) if r else 0)
    # "parameters match the original exactly"
    assert np.array_equal(d.decode(stream), data)
    # hits are exactly the aligned groups that are table members
    members = {tuple(e) for e in d.entries.tolist()}
    want_hits = sum(tuple(data[4 * b:4 * b + 4].tolist()) in members for b in range(nb))
    assert hits == want_hits
    # structure: every 0xFFFF is an escape marker, raw slots are <= 255, codes are 1..K
    codes, esc, tail = _classify(stream)
    assert (codes, esc) == (hits, miss) and tail == (r if r else 0)
    assert int((stream == ESC).sum()) == miss + (1 if r else 0)


@pytest.mark.parametrize("L", [1, 2, 3, 8])
@pytest.mark.parametrize("n", [0, 1, 7, 8, 9, 16, 1000, 4099])
@pytest.mark.parametrize("alphabet,top_k", [(2, 65535), (6, 20), (3, 0)])
def test_round_trip_and_size_identity_other_sequence_lengths(L, n, alphabet, top_k):
    """Listing 2's sequence_length as a parameter: groups, entries and raw runs of L values.  Round
    trip exact, len = H + (1 + L) M + (1 + r if r), hits = aligned groups that are table members,
    and an independent walk of the stream finds the same items."""
    rng = np.random.default_rng(n * 17 + alphabet + 100 * L)
    data = rng.integers(0, alphabet, size=n).astype(np.uint8)
    other = rng.integers(0, alphabet, size=131).astype(np.uint8)
    d = oracle.Dictionary.build([data, other], top_k=top_k, seq=L)
    assert d.seq == L and d.entries.shape[1] == L
    stream, hits, miss = d.encode(data)
    nb, r = divmod(n, L)
    assert hits + miss == nb
    assert stream.size == hits + (1 + L) * miss + ((1 + r) if r else 0)
    assert np.array_equal(d.decode(stream), data)
    members = {tuple(e) for e in d.entries.tolist()}
    assert hits == sum(tuple(data[L * b:L * b + L].tolist()) in members for b in range(nb))
    s, i, codes, esc = stream.tolist(), 0, 0, 0
    while i < len(s):
        if s[i] == ESC:
            assert all(v <= 255 for v in s[i + 1:i + 1 + L])
            esc += 1
            i += 1 + L
        else:
            assert 1 <= s[i] <= d.K
            codes += 1
            i += 1
    assert codes == hits and esc == miss + (1 if r else 0)


def test_closed_forms_other_sequence_lengths():
    data = np.full(4096, 0x5A, dtype=np.uint8)
    for L, n_codes in ((2, 2048), (8, 512)):
        d = oracle.Dictionary.build([data], seq=L)
        assert d.K == 1 and d.entries.tolist() == [[0x5A] * L] and d.counts.tolist() == [4096 - L + 1]
        stream, hits, miss = d.encode(data)
        assert stream.tolist() == [1] * n_codes and miss == 0  # 2 bytes per L weights
    rng = np.random.default_rng(12)
    rnd = rng.integers(0, 256, size=800).astype(np.uint8)
    d0 = oracle.Dictionary.build([rnd], top_k=0, seq=8)
    stream, hits, miss = d0.encode(rnd)
    assert hits == 0 and miss == 100 and stream.size == 900  # every group: marker + 8 values
    assert np.array_equal(stream.reshape(100, 9)[:, 1:].astype(np.uint8).ravel(), rnd)


def test_closed_form_constant_matrix():
    data = np.full(4096, 0x5A, dtype=np.uint8)
    d = oracle.Dictionary.build([data])
    assert d.K == 1 and d.entries.tolist() == [[0x5A] * 4] and d.counts.tolist() == [4093]
    stream, hits, miss = d.encode(data)
    assert stream.tolist() == [1] * 1024 and stream.nbytes == data.size // 2


def test_closed_form_empty_table_all_escapes():
    rng = np.random.default_rng(5)
    data = rng.integers(0, 256, size=400).astype(np.uint8)
    d = oracle.Dictionary.build([data], top_k=0)
    assert d.K == 0
    stream, hits, miss = d.encode(data)
    assert hits == 0 and miss == 100 and stream.size == 500
    assert np.array_equal(stream.reshape(100, 5)[:, 0], np.full(100, ESC, dtype=np.uint16))
    assert np.array_equal(stream.reshape(100, 5)[:, 1:].astype(np.uint8).ravel(), data)


def test_closed_form_all_hit_when_few_distinct():
    rng = np.random.default_rng(6)
    data = rng.integers(0, 6, size=40_000).astype(np.uint8)  # <= 6^4 = 1296 distinct windows
    d = oracle.Dictionary.build([data])
    assert d.n_distinct <= 1296 and d.K == d.n_distinct
    stream, hits, miss = d.encode(data)
    assert miss == 0 and stream.nbytes == data.size // 2  # exactly 4 bits per weight
    assert stream.max() <= d.K and stream.min() >= 1


def test_decoder_rejects_unknown_codes():
    d = oracle.Dictionary.from_entries(np.array([[1, 2, 3, 4]], dtype=np.uint8))
    with pytest.raises(KeyError):
        d.decode(np.array([2], dtype=np.uint16))
    with pytest.raises(KeyError):
        d.decode(np.array([0], dtype=np.uint16))


def test_code_is_rank_plus_one():
    # most frequent aligned group must be coded as 1, next as 2 ...
    data = np.array([9, 9, 9, 9] * 50 + [3, 1, 4, 1] * 20 + [2, 7, 1, 8] * 5, dtype=np.uint8)
    d = oracle.Dictionary.build([data])
    stream, _, _ = d.encode(data)
    # hand count: 9999 x197, 3141 x20, its rotations 1413/4131/1314 x19 each, then 2718 x5
    assert stream[0] == 1 and stream[50] == 2 and stream[70] == 6
    assert d.entries[0].tolist() == [9, 9, 9, 9] and d.counts[:6].tolist() == [197, 20, 19, 19, 19, 5]


# ----------------------------------------------------------------------------
# Quantizers
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("bits", [8, 6, 4, 2, 1])
def test_quantize_paper_end_points_and_error_bound(bits):
    rng = np.random.default_rng(11)
    x = rng.standard_normal(10_000).astype(np.float32) * 0.02
    maxq = 2 ** bits - 1
    q, s, z = oracle.quantize_paper(x, bits=bits)
    assert q[np.argmin(x)] == 0 and q[np.argmax(x)] == maxq and q.max() == maxq
    assert float(s) == float((np.float32(x.max()) - np.float32(x.min())) / np.float32(maxq))
    deq = s.astype(np.float64) * (q.astype(np.float64) - float(z))
    # zero is itself rounded, so the grid may sit up to half a step off x's range at the ends
    assert np.max(np.abs(deq - x)) <= float(s) * (1 + 1e-3) + 1e-9
    inner = (q > 0) & (q < maxq)
    assert np.max(np.abs(deq - x)[inner], initial=0.0) <= 0.5 * float(s) * (1 + 1e-3) + 1e-9
    # levels are a fixed point: quantizing the dequantised values with the same grid returns them
    q2 = np.clip(np.rint(deq / float(s)) + float(z), 0, maxq).astype(np.uint8)
    assert np.array_equal(q, q2)
    with pytest.raises(ValueError):
        oracle.quantize_paper(np.ones(8, dtype=np.float32), bits=bits)


def test_quantize_paper_rejects_other_bit_widths():
    x = np.linspace(-1, 1, 16, dtype=np.float32)
    for bits in (0, 9, -1):
        with pytest.raises(ValueError):
            oracle.quantize_paper(x, bits=bits)
    # halving the bit count keeps every level on the coarser grid's multiples when the ranges nest:
    # x on the integers 0..255 has scale 1 at 8 bits and scale 17 at 4 bits (255 / 15)
    xi = np.arange(256, dtype=np.float32)
    q8, s8, _ = oracle.quantize_paper(xi, bits=8)
    q4, s4, z4 = oracle.quantize_paper(xi, bits=4)
    assert s8 == 1.0 and s4 == 17.0 and z4 == 0.0
    assert np.array_equal(q8, np.arange(256))
    assert np.array_equal(q4, np.rint(xi / 17.0).astype(np.uint8))


def test_quantize_rows_properties():
    rng = np.random.default_rng(12)
    w = (rng.standard_t(5, size=(64, 256)) * 0.02).astype(np.float32)
    w[7] = 0.0
    q, s = oracle.quantize_rows(w)
    assert q.dtype == np.int8 and s[7] == 1.0 and not q[7].any()
    for r in range(64):
        if r == 7:
            continue
        j = int(np.argmax(np.abs(w[r])))
        assert abs(int(q[r, j])) == 127 and np.sign(q[r, j]) == np.sign(w[r, j])
        assert s[r] == np.float32(np.abs(w[r]).max()) / np.float32(127.0)
    assert q.min() >= -127 and q.max() <= 127
    deq = s[:, None].astype(np.float64) * q.astype(np.float64)
    assert np.all(np.abs(deq - w) <= 0.5 * s[:, None] * (1 + 1e-3))
    # hand-worked row: absmax 2.54 -> s = 0.02, values k*0.02 map to k
    row = np.array([[2.54, -2.54, 0.02, -0.04, 0.0, 1.27]], dtype=np.float32)
    q1, s1 = oracle.quantize_rows(row)
    assert q1.tolist() == [[127, -127, 1, -2, 0, 64]] or q1.tolist() == [[127, -127, 1, -2, 0, 63]]


# ----------------------------------------------------------------------------
# Layer product: library fp64 GEMV and closed forms
# ----------------------------------------------------------------------------
def test_layer_forward_against_library_gemv():
    rng = np.random.default_rng(13)
    q = rng.integers(-127, 128, size=(37, 52)).astype(np.int8)
    s = rng.random(37).astype(np.float32) + 0.1
    x = rng.standard_normal((3, 52))
    y = oracle.layer_forward(q, s, x)
    want = (x @ (s[:, None].astype(np.float64) * q.astype(np.float64)).T)
    assert np.allclose(y, want, rtol=1e-13, atol=1e-13)
    # unsigned levels with a zero point (Listing 1's scale * (q - zero))
    qu = rng.integers(0, 256, size=(37, 52)).astype(np.uint8)
    z = rng.integers(0, 256, size=37).astype(np.float32)
    yu = oracle.layer_forward(qu, s, x, zero=z)
    wantu = x @ (s[:, None].astype(np.float64) * (qu.astype(np.float64) - z[:, None])).T
    assert np.allclose(yu, wantu, rtol=1e-13, atol=1e-13)


def test_layer_forward_closed_forms():
    x = np.array([[1.0, -2.0, 3.5, 0.25]])
    ones = np.ones((2, 4), dtype=np.int8)
    s = np.array([0.5, 2.0], dtype=np.float32)
    assert oracle.layer_forward(ones, s, x).tolist() == [[0.5 * 2.75, 2.0 * 2.75]]
    # q == zero everywhere -> output exactly 0
    qz = np.full((2, 4), 9, dtype=np.uint8)
    assert oracle.layer_forward(qz, s, x, zero=np.array([9, 9], dtype=np.float32)).tolist() == [[0.0, 0.0]]
    # a transposed operand would fail this: row r picks x[r]
    eye = np.eye(4, dtype=np.int8)[[2, 0]]
    assert oracle.layer_forward(eye, np.ones(2, dtype=np.float32), x).tolist() == [[3.5, 1.0]]
    # bytes >= 128 are negative when the levels are signed, positive when unsigned
    b = np.array([[0xFF, 0x80, 0x7F, 0x01]], dtype=np.uint8)
    one = np.ones((1, 4))
    assert oracle.layer_forward(b.view(np.int8), np.ones(1, dtype=np.float32), one).tolist() == [[-1 - 128 + 127 + 1]]
    assert oracle.layer_forward(b, np.ones(1, dtype=np.float32), one).tolist() == [[255 + 128 + 127 + 1]]
