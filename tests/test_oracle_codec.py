"""Pins of the CPU oracle's whole encode/decode: an independent numpy reader of the packed
format (explicit Hadamard matrix, float64), the size accounting printed in Sec. 3.4, the special
cases tau = 0 / tau = inf, closed forms for one-hot tiles, error bounds and direction-only sanity."""
import math
import os

import numpy as np
import pytest
import scipy.linalg
import torch

import oracle as O
from paper_2506_01352_b200 import synth
from tests.test_oracle_steps import read_golden


# --------------------------------------------------------------------------------------
# An independent reader of the packed format, written from the format description only.
# --------------------------------------------------------------------------------------

def parse(packed: np.ndarray):
    b = packed.tobytes()
    u32 = lambda o: int.from_bytes(b[o:o + 4], "little")
    u64 = lambda o: int.from_bytes(b[o:o + 8], "little")
    h = dict(magic=b[0:4], version=u32(4), dtype=u32(8), rounding=u32(12), tokens=u64(16), hidden=u32(24),
             tile=u32(28), group_tokens=u32(32), budget=u32(36), n_tiles=u64(64), payload_bytes=u64(72),
             total_bytes=u64(80))
    al = lambda x: (x + 127) // 128 * 128
    n = h["n_tiles"]
    o_bm = 128
    o_sz = al(o_bm + (n + 7) // 8)
    o_pv = al(o_sz + 4 * n)
    o_pl = al(o_pv + n)
    bits = np.unpackbits(packed[o_bm:o_bm + (n + 7) // 8], bitorder="little")[:n]
    sz = packed[o_sz:o_sz + 4 * n].view(np.float16).reshape(n, 2).astype(np.float64)
    pv = packed[o_pv:o_pv + n]
    h.update(is_hi=bits, scale=sz[:, 0], zero=sz[:, 1], pivot=pv, off_payload=o_pl,
             sections=(o_bm, o_sz, o_pv, o_pl))
    return h


def reference_decode(packed: np.ndarray) -> np.ndarray:
    """float64 decode with an explicit Sylvester matrix; agrees with the codec to rounding."""
    h = parse(packed)
    G, n = h["tile"], h["n_tiles"]
    lo = h["budget"] // 1000
    width = lo + h["is_hi"].astype(np.int64)
    stream = np.unpackbits(packed[h["off_payload"]:h["off_payload"] + h["payload_bytes"]], bitorder="little")
    H = scipy.linalg.hadamard(G).astype(np.float64) / math.sqrt(G)
    out = np.empty((n, G))
    pos = 0
    for t in range(n):
        w = int(width[t])
        codes = stream[pos:pos + G * w].reshape(G, w) @ (1 << np.arange(w))
        pos += G * w
        v = h["zero"][t] + codes * h["scale"][t]
        if h["pivot"][t] & 0x80:
            d = h["pivot"][t] & 0x7F
            v = v @ H.T
            v[[0, d]] = v[[d, 0]]
        out[t] = v
    assert pos == 8 * h["payload_bytes"]
    return out.reshape(h["tokens"], h["hidden"])


def tiny(seed=0, dtype=O.F32):
    x = synth.make("c1_tiny", microbatch=seed)
    if dtype == O.BF16:
        x = x.to(torch.bfloat16)
    return synth.to_host_array(x)


def relerr(y, x):
    y = np.asarray(y, np.float64); x = np.asarray(x, np.float64)
    return float(((y - x) ** 2).sum() / (x ** 2).sum())


def bf16_to_f32(a):
    return (a.astype(np.uint32) << 16).view(np.float32)


# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("G", [32, 64])
@pytest.mark.parametrize("beta", [3000, 3800, 4000])
def test_format_invariants_and_independent_decode(G, beta):
    x = tiny()
    p = O.Params(tokens=128, hidden=256, group_tokens=64, tile=G, budget_millibits=beta)
    packed = O.encode(p, x)
    L = O.layout(p)
    h = parse(packed)
    assert h["magic"] == b"TAHQ" and h["version"] == 1 and h["tile"] == G and h["group_tokens"] == 64
    assert packed.size == L["total_bytes"] == h["total_bytes"] == O.packed_bound(p)
    assert h["sections"] == (L["off_bitmap"], L["off_scale_zero"], L["off_pivot"], L["off_payload"])
    ng = L["tiles_per_group"]
    k_hi = ng * (beta % 1000) // 1000
    per_group = h["is_hi"].reshape(-1, ng).sum(axis=1)
    assert (per_group == k_hi).all()                                     # exactly top-p% per sample
    payload_bits = G * (h["n_tiles"] * (beta // 1000) + per_group.sum())
    assert payload_bits == 8 * h["payload_bytes"]
    assert payload_bits <= beta * x.size // 1000 < payload_bits + G * L["n_groups"] + 1   # budget met, never exceeded
    y = O.decode(p, packed)
    ref = reference_decode(packed)
    step = h["scale"].max()
    assert np.abs(y - ref).max() <= 1e-5 * max(step, 1.0) + 1e-6 * np.abs(ref).max()
    assert relerr(y, x) < 0.2                                            # squared relative error; sanity only


def test_bits_per_element_against_the_papers_accounting():
    g = read_golden("paper_sec3_4_size.txt")
    G = int(g["tile"])
    p = O.Params(tokens=4096, hidden=4096, group_tokens=1024, tile=G,
                 budget_millibits=int(round(3000 + 1000 * float(g["int4_fraction"]))))
    L = O.layout(p)
    n = p.tokens * p.hidden
    payload_bits = 8 * L["payload_bytes"] / n
    assert 0 <= 3.8 - payload_bits < 1e-4                                 # 80% INT4 + 20% INT3
    meta_bits = 8 * (L["total_bytes"] - L["payload_bytes"]) / n
    # 16 (scale) + 16 (zero) + 1 (bit map) + 8 (pivot byte) = 41 bits per 64-wide tile; the paper's
    # 0.61 corresponds to 39 bits (a 6-bit pivot index)
    assert abs(meta_bits - 41 / 64) < 1e-3
    assert abs(meta_bits - float(g["metadata_bits_per_element"])) < 0.04
    assert abs(payload_bits + meta_bits - float(g["bits_per_element"])) < 0.04


def test_packed_bound_closed_form():
    for (T, Cc, S, G, beta) in [(128, 256, 64, 64, 3800), (8192, 768, 1024, 64, 3000), (77, 96, 11, 32, 2200),
                                (5, 128, 0, 128, 7500), (16, 64, 4, 8, 2000)]:
        p = O.Params(tokens=T, hidden=Cc, group_tokens=S, tile=G, budget_millibits=beta)
        S2 = S or T
        n = T * Cc // G
        ng = S2 * Cc // G
        payload = (T // S2) * (G // 8) * (ng * (beta // 1000) + ng * (beta % 1000) // 1000)
        al = lambda v: (v + 127) // 128 * 128
        want = al(al(al(al(128 + (n + 7) // 8) + 4 * n) + n) + payload)
        assert O.packed_bound(p) == want
    bad = [dict(tile=48), dict(hidden=100), dict(group_tokens=5), dict(budget_millibits=1999),
           dict(budget_millibits=8001), dict(tile=256), dict(dtype=2)]
    for kw in bad:
        base = dict(tokens=128, hidden=256, group_tokens=64, tile=64, budget_millibits=3800)
        base.update(kw)
        assert O.packed_bound(O.Params(**base)) == 0


def test_tau_inf_integer_budget_is_plain_group_quantisation():
    # Sec. 3.3 / App. tau: never transforming + one width = textbook per-group min-max quantisation
    x = tiny(1)
    for bits in (3, 4, 8):
        p = O.Params(tokens=128, hidden=256, group_tokens=64, tile=64, budget_millibits=1000 * bits,
                     tau=float("inf"))
        packed = O.encode(p, x)
        assert not parse(packed)["pivot"].any() and not parse(packed)["is_hi"].any()
        y = O.decode(p, packed)
        t = x.reshape(-1, 64)
        qmax = np.float32(2 ** bits - 1)
        z = t.min(axis=1, keepdims=True).astype(np.float16).astype(np.float32)
        s = ((t.max(axis=1, keepdims=True) - z) / qmax).astype(np.float16).astype(np.float32)
        q = np.clip(np.rint((t - z).astype(np.float64) * (np.float32(1) / s).astype(np.float64)), 0, qmax)
        want = (q.astype(np.float64) * s.astype(np.float64) + z.astype(np.float64)).astype(np.float32)  # one rounding
        assert np.array_equal(y.reshape(-1, 64), want)


def test_tau_zero_transforms_every_nonzero_tile():
    x = tiny(2).copy()
    x.reshape(-1, 64)[7] = 0
    p = O.Params(tokens=128, hidden=256, group_tokens=64, budget_millibits=4000, tau=0.0)
    pv = parse(O.encode(p, x))["pivot"]
    assert pv[7] == 0 and (np.delete(pv, 7) & 0x80).all()
    d = pv & 0x7F
    want = np.abs(x.reshape(-1, 64)).argmax(axis=1)
    assert np.array_equal(np.delete(d, 7), np.delete(want, 7))


@pytest.mark.parametrize("beta", [2000, 3000, 3800, 8000])
def test_one_hot_tiles_round_trip_in_closed_form(beta):
    # a lone spike is flagged, becomes a constant tile, and comes back exactly (v/8 fits binary16 here)
    x = np.zeros((8, 256), np.float32)
    vals = [8.0, -24.0, 1000.0, 0.5, -4096.0, 3.0, 20.0, 2 ** -3]
    for i, v in enumerate(vals):
        x[i, 64 * (i % 4) + (5 * i + 1) % 64] = v
    p = O.Params(tokens=8, hidden=256, group_tokens=8, budget_millibits=beta)
    packed = O.encode(p, x)
    h = parse(packed)
    tiles = [4 * i + (i % 4) for i in range(8)]
    assert all(h["pivot"][t] == 0x80 | ((5 * i + 1) % 64) for i, t in enumerate(tiles))
    assert all(h["scale"][t] == 0 for t in tiles)                       # range of a constant tile
    assert np.array_equal(O.decode(p, packed), x)


def test_scale_does_not_depend_on_the_outlier_magnitude():
    # Sec. 3.3: once the pivot is moved to coordinate 0 it only shifts every output by the same
    # amount, so the range (hence the scale) is that of the rest of the tile
    rng = np.random.default_rng(3)
    base = rng.integers(-8, 9, 64).astype(np.float32)
    scales = []
    for v in (64.0, 512.0, 4096.0):
        x = base.copy(); x[37] = v
        p = O.Params(tokens=1, hidden=64, budget_millibits=4000)
        h = parse(O.encode(p, x))
        assert h["pivot"][0] == 0x80 | 37
        scales.append(h["scale"][0])
    # equal up to the binary16 rounding of the zero-point (its ulp grows with the shift)
    assert max(scales) - min(scales) <= 0.02 * min(scales)
    unflagged = parse(O.encode(O.Params(tokens=1, hidden=64, budget_millibits=4000, tau=float("inf")),
                               np.where(np.arange(64) == 37, np.float32(4096), base)))["scale"][0]
    assert unflagged > 20 * scales[0]


def test_eight_bits_is_near_lossless_and_error_falls_with_width():
    x = tiny(3)
    errs = []
    for beta in (2000, 3000, 4000, 6000, 8000):
        p = O.Params(tokens=128, hidden=256, group_tokens=64, budget_millibits=beta)
        errs.append(relerr(O.decode(p, O.encode(p, x)), x))
    assert errs == sorted(errs, reverse=True)
    assert errs[-1] < 1e-4                                              # relative L2 error < 1%
    assert all(e < 1 for e in errs)                                     # contraction (Assumption 4.4)


def test_direction_only_sanity_on_outlier_data():
    # App. tau and App. bit sweep give directions only: transform on < off; mixed widths lie between
    x = tiny(4)
    def err(**kw):
        p = O.Params(tokens=128, hidden=256, group_tokens=64, **kw)
        return relerr(O.decode(p, O.encode(p, x)), x)
    assert err(budget_millibits=3800, tau=2.0) < err(budget_millibits=3800, tau=float("inf"))
    assert err(budget_millibits=4000) < err(budget_millibits=3800) < err(budget_millibits=3000)


def test_per_coordinate_error_bound():
    x = tiny(5)
    p = O.Params(tokens=128, hidden=256, group_tokens=64, budget_millibits=3800)
    packed = O.encode(p, x)
    h = parse(packed)
    y = O.decode(p, packed).reshape(-1, 64).astype(np.float64)
    t = x.reshape(-1, 64).astype(np.float64)
    s = h["scale"]
    flagged = (h["pivot"] & 0x80) != 0
    # untransformed tiles: every coordinate within half a step (plus binary16 rounding of z, s)
    width = 3 + h["is_hi"]
    slack = 2.0 ** -10 * (np.abs(t).max(axis=1) + s * (2.0 ** width))
    assert (np.abs(y - t).max(axis=1)[~flagged] <= (s / 2 + slack)[~flagged]).all()
    # transformed tiles: the inverse is orthonormal, so the L2 error is at most sqrt(G) half-steps
    l2 = np.sqrt(((y - t) ** 2).sum(axis=1))
    assert (l2[flagged] <= (8 * (s / 2 + slack))[flagged]).all()
    assert flagged.any() and (~flagged).any()


def test_bf16_tensor_path():
    xb = tiny(6, O.BF16)
    p = O.Params(tokens=128, hidden=256, group_tokens=64, dtype=O.BF16, budget_millibits=3800)
    packed = O.encode(p, xb)
    # a bf16 tensor encodes exactly like the same values held in fp32 (the widening is exact)
    pf = O.Params(tokens=128, hidden=256, group_tokens=64, dtype=O.F32, budget_millibits=3800)
    packed_f = O.encode(pf, bf16_to_f32(xb))
    assert np.array_equal(packed[128:], packed_f[128:])
    y = O.decode(p, packed)
    yf = O.decode(pf, packed_f)
    want = torch.from_numpy(yf).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(y, want)                                       # round-to-nearest-even narrowing


def test_groups_are_ranked_independently_and_threads_do_not_matter():
    x = tiny(7)
    p = O.Params(tokens=128, hidden=256, group_tokens=64, budget_millibits=3500)
    O.set_threads(1)
    a = O.encode(p, x)
    O.set_threads(os.cpu_count() or 2)
    b = O.encode(p, x)
    assert np.array_equal(a, b)
    # encoding one sample alone gives the same bit map as that sample inside the batch
    p1 = O.Params(tokens=64, hidden=256, group_tokens=64, budget_millibits=3500)
    solo = parse(O.encode(p1, x[64:]))["is_hi"]
    assert np.array_equal(parse(a)["is_hi"][256:], solo)
    # with group_tokens = 0 the whole tensor is one ranking group
    p0 = O.Params(tokens=128, hidden=256, group_tokens=0, budget_millibits=3500)
    assert parse(O.encode(p0, x))["is_hi"].sum() == 512 * 500 // 1000


def test_decode_rejects_a_foreign_header():
    x = tiny(8)
    p = O.Params(tokens=128, hidden=256, group_tokens=64)
    packed = O.encode(p, x)
    bad = packed.copy(); bad[0] ^= 1
    with pytest.raises(RuntimeError):
        O.decode(p, bad)
    with pytest.raises(RuntimeError):
        O.decode(O.Params(tokens=128, hidden=256, group_tokens=64, budget_millibits=3000), packed)


def test_stochastic_mode_whole_tensor_is_unbiased():
    x = tiny(9)[:16]
    acc = np.zeros_like(x, dtype=np.float64)
    n = 300
    for seed in range(n):
        p = O.Params(tokens=16, hidden=256, group_tokens=16, budget_millibits=3000, rounding=1, seed=seed,
                     tau=float("inf"))
        acc += O.decode(p, O.encode(p, x))
    p0 = O.Params(tokens=16, hidden=256, group_tokens=16, budget_millibits=3000, tau=float("inf"))
    det = O.decode(p0, O.encode(p0, x))
    assert relerr(acc / n, x) < 0.1 * relerr(det, x)


# ---------------------------------------------------------------- allocation tiles wider than quantisation tiles (Sec. 3.2)
def _shannon64(v):
    a = np.abs(v.astype(np.float64))
    p = a / (a.sum() + 1e-8)
    return float(-(p * np.log2(p + 1e-8)).sum())


def _bitmap(p, buf):
    L = O.layout(p)
    return np.unpackbits(buf[L["off_bitmap"]:L["off_bitmap"] + (L["n_tiles"] + 7) // 8], bitorder="little")[:L["n_tiles"]]


def test_tree_sum_of_any_length():
    """A partial sum without a neighbour waits for the next level: n = 3 -> (x0+x1)+x2, n = 6 -> ((x0+x1)+(x2+x3))+(x4+x5)."""
    f = np.float32
    x = np.array([1e8, 1.0, -1e8, 3.0, 5.0, 7.0], dtype=np.float32)
    assert O.treesum(x[:3]) == f(f(x[0] + x[1]) + x[2])
    assert O.treesum(x) == f(f(f(x[0] + x[1]) + f(x[2] + x[3])) + f(x[4] + x[5]))
    y = np.arange(1, 13, dtype=np.float32)
    assert O.treesum(y) == 78.0
    # 768 = 3 * 256: three power-of-two blocks, ((b0 + b1) + b2)
    z = np.random.default_rng(1).standard_normal(768).astype(np.float32)
    b = [O.treesum(z[i * 256:(i + 1) * 256]) for i in range(3)]
    assert O.treesum(z) == f(f(b[0] + b[1]) + b[2])


@pytest.mark.parametrize("hidden,G,A", [(256, 64, 128), (256, 64, 256), (768, 64, 192), (768, 64, 768), (512, 32, 128)])
def test_allocation_tile_wider_than_quantisation_tile(hidden, G, A):
    """A = m*G: the entropy is taken over A channels, the top-p% of the S*C/A allocation tiles of a sample get
    the higher width, and all m quantisation tiles inside share it; A = C is token-level allocation."""
    rng = np.random.default_rng(hidden + A)
    S, B = 16, 3
    x = (rng.standard_normal((B * S, hidden)) * np.exp(rng.standard_normal((B * S, 1)))).astype(np.float32)
    x[:, ::53] *= 20
    p = O.Params(tokens=B * S, hidden=hidden, group_tokens=S, tile=G, budget_millibits=3500, alloc_tile=A)
    L = O.layout(p)
    m, na_g = A // G, S * (hidden // A)
    k_a = na_g * 500 // 1000
    assert L["k_hi"] == k_a * m
    assert L["payload_bytes"] == B * (G // 8) * (L["tiles_per_group"] * 3 + L["k_hi"])
    buf = O.encode(p, x)
    bm = _bitmap(p, buf).reshape(B, na_g, m)
    assert (bm.min(axis=2) == bm.max(axis=2)).all()                 # one width per allocation tile
    assert (bm[:, :, 0].sum(axis=1) == k_a).all()                   # exactly the top-p% per sample
    # which ones: the float64 Shannon entropy over A channels, wherever the ranking is not a near-tie
    tiles = x.reshape(B, na_g, A)
    for b in range(B):
        h = np.array([_shannon64(t) for t in tiles[b]])
        order = np.argsort(-h, kind="stable")
        if k_a and k_a < na_g and h[order[k_a - 1]] - h[order[k_a]] > 1e-4:
            assert set(np.flatnonzero(bm[b, :, 0])) == set(order[:k_a])
    # decode still inverts it, and the header tells the two apart
    y = O.decode(p, buf)
    assert np.abs(y - x).max() <= np.abs(x).max()
    assert int(buf[88:92].view(np.uint32)[0]) == A


def test_default_allocation_tile_is_the_quantisation_tile():
    x = np.random.default_rng(5).standard_normal((32, 256)).astype(np.float32)
    a = O.encode(O.Params(tokens=32, hidden=256, group_tokens=16, tile=64, budget_millibits=3800), x)
    b = O.encode(O.Params(tokens=32, hidden=256, group_tokens=16, tile=64, budget_millibits=3800, alloc_tile=64), x)
    assert np.array_equal(a, b)
    for bad in (96, 48, 512):
        assert O.packed_bound(O.Params(tokens=32, hidden=256, group_tokens=16, tile=64, alloc_tile=bad)) == 0
