"""Pins of the oracle's FP8 (E4M3) page quantiser: the code table against torch's float8_e4m3fn, the
rounding against brute force over that table (nearest, ties to the even code, saturation at 448),
the power-of-two page scales, and the append rule."""
import numpy as np
import pytest
import torch

from helpers import Problem
from oracle import oracle as orc


def table():
    codes = np.arange(256, dtype=np.uint8)
    vals = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    return codes, vals


def test_code_table_is_e4m3fn():
    codes, vals = table()
    dec = orc.fp8_decode(codes)
    assert np.isnan(dec[[0x7f, 0xff]]).all() and np.isnan(vals[[0x7f, 0xff]]).all()
    ok = ~np.isnan(vals)
    assert (dec[ok] == vals[ok]).all()
    assert dec[0x7e] == 448.0 and dec[0x01] == 2.0 ** -9 and dec[0x08] == 2.0 ** -6 and dec[0x38] == 1.0
    assert (orc.fp8_encode(dec[ok]) == codes[ok]).all() or set(codes[ok][orc.fp8_encode(dec[ok]) != codes[ok]]) <= {0x80}


def test_rounding_is_nearest_even_with_saturation():
    codes, vals = table()
    pos = np.array([c for c in codes if c < 0x7f], np.uint8)            # non-negative finite codes, ascending in value
    pv = vals[pos]
    rng = np.random.default_rng(5)
    y = np.concatenate([rng.uniform(-460, 460, 4000), rng.normal(0, 1, 4000), rng.normal(0, 0.01, 2000),
                        (pv[:-1] + pv[1:]) / 2, -(pv[:-1] + pv[1:]) / 2, pv, [0.0, 448.0, 449.0, 1e9, -1e9, 2.0 ** -10, 2.0 ** -11]])
    got = orc.fp8_encode(y)
    for yi, gi in zip(y, got):
        a = abs(yi)
        dist = np.abs(pv - min(a, 448.0))
        best = np.flatnonzero(dist == dist.min())
        want = pos[best[0]] if len(best) == 1 else [c for c in pos[best] if c % 2 == 0][0]    # tie: even mantissa
        want |= 0x80 if yi < 0 else 0
        assert gi == want, (yi, gi, want)
    inr = np.abs(y) <= 448
    t = torch.from_numpy(y[inr]).to(torch.float32).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    f32 = y[inr].astype(np.float32).astype(np.float64)                 # torch rounds the fp32 value
    assert (orc.fp8_encode(f32) == t).all() or set(np.flatnonzero(orc.fp8_encode(f32) != t)) <= set(np.flatnonzero(f32 == 0))


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_page_scales_and_dequantised_error(dtype):
    pb = Problem(41, N=2, Hq=4, Hkv=2, d=32, B=4, g=8, kv_lens=(61, 16), dtype=dtype, scale=3.0)
    sh = pb.sh
    kc, vc, ks, vs = orc.fp8_quantize_pages(sh, pb.kv)
    for s in range(2):
        L = (61, 16)[s]
        for p in range(pb.pages(s)):
            ph = pb.page_table[s, p]
            n = min(8, L - 8 * p)
            for kh in range(2):
                for codes, scales, X in ((kc, ks, pb.K[s]), (vc, vs, pb.V[s])):
                    x = X[8 * p:8 * p + n, kh].astype(np.float64)
                    sc = float(scales[ph, kh])
                    e = np.log2(sc)
                    assert e == round(e) and -6 <= e <= 7
                    amax = np.abs(x).max()
                    assert amax <= 448 * sc and (e == -6 or amax > 448 * sc / 2)        # the smallest such power of two
                    deq = sc * orc.fp8_decode(codes[ph, kh, :n])
                    assert (np.abs(deq - x) <= np.maximum(2.0 ** -4 * np.abs(x), sc * 2.0 ** -10)).all()
                    assert (codes[ph, kh, n:] == 0).all()
                    assert (orc.fp8_encode(deq / sc) == codes[ph, kh, :n]).all()       # re-quantising is the identity


def test_append_requantises_touched_pages_from_old_and_new_rows():
    pb = Problem(42, N=2, Hq=4, Hkv=2, d=16, B=6, g=4, kv_lens=(10, 8), extra_pages=3, dtype="bf16")
    sh = pb.sh
    kc, vc, ks, vs = orc.fp8_quantize_pages(sh, pb.kv)
    kb = pb.rand_elem((2, 6, 2, 16), scale=6.0)                          # larger than the cache: scales must grow
    vb = pb.rand_elem((2, 6, 2, 16), scale=0.2)
    kv_len = pb.kv_len.copy()
    kc2, vc2, ks2, vs2 = kc.copy(), vc.copy(), ks.copy(), vs.copy()
    orc.fp8_append_block(sh, pb.page_table, kv_len, kc2, vc2, ks2, vs2, kb, vb)
    assert kv_len.tolist() == [16, 14]
    kbf, vbf = pb.f(kb).astype(np.float64), pb.f(vb).astype(np.float64)
    for s, L0 in enumerate((10, 8)):
        for p in range(L0 // 4, (L0 + 6 - 1) // 4 + 1):
            ph = pb.page_table[s, p]
            n_old = max(0, L0 - 4 * p)
            rows = range(4 * p + n_old - L0, min(L0 + 6, 4 * p + 4) - L0)
            for kh in range(2):
                for old_c, old_s, new_c, new_s, blk in ((kc, ks, kc2, ks2, kbf), (vc, vs, vc2, vs2, vbf)):
                    x = np.concatenate([float(old_s[ph, kh]) * orc.fp8_decode(old_c[ph, kh, :n_old]), blk[s, list(rows), kh]])
                    e = -6
                    while e < 7 and np.abs(x).max() > 448 * 2.0 ** e:
                        e += 1
                    assert new_s[ph, kh] == 2.0 ** e
                    assert (new_c[ph, kh, :len(x)] == orc.fp8_encode(x / 2.0 ** e)).all()
                    assert (new_c[ph, kh, len(x):] == 0).all()
    # pages before the first touched one are untouched
    for s, L0 in enumerate((10, 8)):
        for p in range(L0 // 4):
            ph = pb.page_table[s, p]
            assert (kc2[ph] == kc[ph]).all() and (ks2[ph] == ks[ph]).all()
    # dequantised pool: exact in bf16, and equal to scale * table value
    orc.fp8_dequantize_pages(sh, kc2, vc2, ks2, vs2, orc.KV(sh, pb.k_pages, pb.v_pages, pb.kmin, pb.kmax, pb.page_table, kv_len))
    ph = pb.page_table[0, 3]
    assert (pb.f(pb.k_pages)[ph, 1, :4].astype(np.float64) == float(ks2[ph, 1]) * orc.fp8_decode(kc2[ph, 1, :4])).all()
