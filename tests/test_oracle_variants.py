"""Pins for the oracle's parameterisation variants (CPU only): the 8-bit e4m3 conversions, the Llama-3.1 rescaled
frequency table, and rotation of only the first R coordinates of a head.

Each test checks the oracle against something that is not the oracle's own formula: the format's definition
written out as a table, torch's float8 cast (a library routine), the regions of the rescaling rule that have a
closed form, the rope-scaling routine of the transformers library, and reduction of the partial rotation to the
full rotation that tests/test_oracle_rope.py pins.
"""
import math

import numpy as np
import pytest
import torch


# ------------------------------------------------------------------------------------------------ e4m3
def e4m3_table():
    """All 256 codes decoded from the format's definition: sign, 4 exponent bits with bias 7, 3 mantissa bits;
    exponent field 0 is subnormal (m * 2^-9); code 0x7f / 0xff is NaN."""
    out = np.empty(256, np.float64)
    for c in range(256):
        e, m = (c >> 3) & 15, c & 7
        if e == 15 and m == 7:
            v = math.nan
        elif e == 0:
            v = m * 2.0**-9
        else:
            v = (1 + m / 8) * 2.0 ** (e - 7)
        out[c] = -v if c & 0x80 else v
    return out


def test_e4m3_decode_is_the_format_table_and_encode_inverts_it(oracle_mod):
    table = e4m3_table()
    got = oracle_mod.e4m3_to_double(np.arange(256, dtype=np.uint8))
    assert np.array_equal(np.isnan(got), np.isnan(table)) and np.array_equal(got[~np.isnan(table)], table[~np.isnan(table)])
    assert table[0x7E] == 448.0 and table[0x08] == 2.0**-6 and table[0x01] == 2.0**-9
    finite = np.array([c for c in range(256) if not math.isnan(table[c])], np.uint8)
    assert np.array_equal(oracle_mod.e4m3_from_double(table[finite]), finite)  # -0.0 keeps its sign too
    assert np.all(np.diff(table[:0x7F]) > 0)  # positive codes are ordered like their values


def test_e4m3_rounding_is_to_nearest_with_ties_to_even_and_saturates(oracle_mod):
    table = e4m3_table()
    pos = table[:0x7F]
    for c in range(0x7E):
        a, b = pos[c], pos[c + 1]
        mid = (a + b) / 2
        even = c if c % 2 == 0 else c + 1
        below, above = np.nextafter(mid, a), np.nextafter(mid, b)
        assert oracle_mod.e4m3_from_double(np.array([mid, below, above])).tolist() == [even, c, c + 1]
        assert oracle_mod.e4m3_from_double(np.array([-mid, -below, -above])).tolist() == [even | 0x80, c | 0x80, (c + 1) | 0x80]
    big = np.array([448.0, np.nextafter(448.0, 1e9), 463.9, 464.0, 1e30, np.inf, -449.0, -np.inf])
    assert oracle_mod.e4m3_from_double(big).tolist() == [0x7E] * 6 + [0xFE] * 2
    assert oracle_mod.e4m3_from_double(np.array([np.nan]))[0] == 0x7F


def test_e4m3_matches_torch_float8_cast(oracle_mod):
    # torch's cast is a one-step round-to-nearest-even from float32 (it does not saturate, so stay below 464)
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(200_000) * 3, rng.standard_normal(100_000) * 0.01, rng.uniform(-463, 463, 100_000),
                        rng.uniform(-2.0**-5, 2.0**-5, 100_000)]).astype(np.float32)  # fmt: skip
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = oracle_mod.e4m3_from_double(x.astype(np.float64))
    assert np.array_equal(got, want)


def bf16_bits_to_f32(bits_: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits_).view(np.int16)).view(torch.bfloat16).float()


def torch_e4m3(x32: torch.Tensor) -> np.ndarray:
    """float32 -> e4m3 codes by torch's cast (one step, nearest even), saturating first as the cache-write kernels do."""
    return x32.clamp(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8).numpy()


@pytest.mark.parametrize("k_scale,v_scale", [(0.3, 0.0173), (2.7, 0.3), (0.0173, 2.7), (0.5, 0.25)])
def test_e4m3_cache_codes_follow_the_engine_rule_at_any_scale(oracle_mod, k_scale, v_scale):
    """The code of an 8-bit cache element is e4m3(binary32(bf16 value) / scale): the bf16 key or value a bf16 cache would
    hold, an IEEE binary32 division by the per-tensor scale, one rounding to e4m3.  Pinned against torch (bf16 -> float32,
    float32 division, float8 cast) at scales whose reciprocal is not a binary32 number; quantising the unrounded
    rotated key instead of its bf16 value is a visibly different rule on these inputs."""
    rng = np.random.default_rng(21)
    kb, vb = small_store(rng, L=2, T=64, H=2, D=32)
    lens = np.array([16, 16, 16, 16], np.int32)
    offs = np.array([0, 16, 32, 48], np.int64)
    table = np.arange(8, dtype=np.int32)
    res = oracle_mod.inject([2, 0, 3, 1], offs, lens, kb, vb, 1e4, 3, table, 16, 8, k_scale=k_scale, v_scale=v_scale)
    ks, vs = torch.tensor(k_scale, dtype=torch.float32), torch.tensor(v_scale, dtype=torch.float32)
    want_k = torch_e4m3(bf16_bits_to_f32(res.k_bf16) / ks)
    want_v = torch_e4m3(bf16_bits_to_f32(res.v) / vs)
    assert np.array_equal(res.k_fp8, want_k) and np.array_equal(res.v_fp8, want_v)
    unrounded_k = torch_e4m3(torch.from_numpy(res.k_ref).float() / ks)
    assert (unrounded_k != want_k).any()


@pytest.mark.parametrize("scale", [0.3, 2.7, 0.9, 0.0173])
def test_e4m3_division_rule_on_every_bf16_value(oracle_mod, scale):
    """All finite bf16 values as the values of one long fact: the codes are those of torch's float32 division and float8
    cast.  At 0.3, 2.7 and 0.9 a product with the rounded reciprocal would give other codes for some of these values,
    so the pin tells division from multiplication; large quotients saturate at +-448."""
    every = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    x = bf16_bits_to_f32(every)
    every = every[torch.isfinite(x).numpy()]
    x = bf16_bits_to_f32(every)
    n = every.size // 2
    store = np.ascontiguousarray(every[: 2 * n].reshape(1, n, 1, 2))  # one layer, one head of two coordinates per token
    nb = (n + 15) // 16
    res = oracle_mod.inject([0], np.array([0], np.int64), np.array([n], np.int32), store, store, 1e4, 0,
                            np.arange(nb, dtype=np.int32), 16, nb, k_scale=1.0, v_scale=scale)  # fmt: skip
    st = torch.tensor(scale, dtype=torch.float32)
    want = torch_e4m3(x[: 2 * n] / st).reshape(1, n, 1, 2)
    assert np.array_equal(res.v_fp8, want)
    by_product = torch_e4m3(x[: 2 * n] * (1.0 / st)).reshape(1, n, 1, 2)
    if scale != 0.0173:
        assert (by_product != want).any()
    big = (x[: 2 * n].abs() / st > 470).numpy().reshape(1, n, 1, 2)
    assert big.any() and set(res.v_fp8[big].tolist()) <= {0x7E, 0xFE}


# ------------------------------------------------------------------------------------------------ rescaled frequencies
def test_llama3_table_regions_with_closed_forms(oracle_mod):
    for R, theta in ((128, 5e5), (64, 1e4)):
        plain64 = np.array([theta ** (-(2 * i) / R) for i in range(R // 2)])
        got = oracle_mod.inv_freq_llama3(R, theta, factor=8.0, low_freq_factor=1.0, high_freq_factor=4.0, original_max=8192.0)
        wavelen = 2 * math.pi / plain64
        keep, slow = wavelen < 8192 / 4, wavelen > 8192 / 1
        assert keep.any() and slow.any() and (~keep & ~slow).any()  # all three regions occur
        assert np.array_equal(got[keep], oracle_mod.inv_freq(R, theta)[keep])  # short wavelengths: untouched, bit for bit
        assert np.array_equal(got[slow], (plain64[slow] / 8).astype(np.float32))  # long wavelengths: slowed by the factor
        mid = ~keep & ~slow
        assert np.all(got[mid] < plain64[mid]) and np.all(got[mid] > plain64[mid] / 8)
        assert np.all(np.diff(got.astype(np.float64)) < 0)  # still a decreasing table
        # the blend is continuous at both ends: a pair just inside the band is close to the rule outside it
        lo_edge = oracle_mod.inv_freq_llama3(2, 1.0, 8.0, 1.0, 4.0, 2 * math.pi * 0.999999)  # f = 1, wavelength just above max/low
        assert lo_edge[0] == np.float32(1 / 8)
    # factor 1 changes nothing
    assert np.array_equal(oracle_mod.inv_freq_llama3(128, 5e5, factor=1.0), oracle_mod.inv_freq(128, 5e5))


def test_llama3_table_matches_the_transformers_routine(oracle_mod):
    rope_utils = pytest.importorskip("transformers.modeling_rope_utils")
    fn = rope_utils.ROPE_INIT_FUNCTIONS.get("llama3")
    if fn is None:
        pytest.skip("this transformers build has no llama3 rope initialiser")
    from transformers import LlamaConfig

    params = {"rope_type": "llama3", "factor": 8.0, "low_freq_factor": 1.0, "high_freq_factor": 4.0,
              "original_max_position_embeddings": 8192, "rope_theta": 500000.0}  # fmt: skip
    try:
        cfg = LlamaConfig(hidden_size=4096, num_attention_heads=32, rope_theta=500000.0, rope_scaling=dict(params),
                          rope_parameters=dict(params), max_position_embeddings=131072)  # fmt: skip
        inv, _ = fn(cfg, "cpu")
    except Exception as e:  # the config surface of this library changes between releases
        pytest.skip(f"transformers rope initialiser not callable this way: {e}")
    got = oracle_mod.inv_freq_llama3(128, 5e5)
    # the library computes in float32: agreement to a few float32 ulps
    assert np.allclose(inv.double().numpy(), got.astype(np.float64), rtol=2e-6, atol=0)


# ------------------------------------------------------------------------------------------------ partial rotary
@pytest.mark.parametrize("style", [0, 1])
def test_partial_rotation_reduces_to_the_full_rotation_of_the_leading_block(oracle_mod, style):
    rng = np.random.default_rng(7)
    D, R, theta = 64, 32, 1e4
    x = rng.standard_normal((50, D))
    pos = rng.integers(0, 100_000, 50)
    y = oracle_mod.rope_rows(x, pos, theta, style=style, rotary_dim=R)
    assert np.array_equal(y[:, R:], x[:, R:])  # the tail is copied
    # the leading block is an R-dimensional head of its own (frequencies theta^(-2i/R), pairs inside the block)
    assert np.array_equal(y[:, :R], oracle_mod.rope_rows(x[:, :R].copy(), pos, theta, style=style))
    # R = D is the plain rotation
    assert np.array_equal(oracle_mod.rope_rows(x, pos, theta, style=style, rotary_dim=D), oracle_mod.rope_rows(x, pos, theta, style=style))
    assert not np.array_equal(y[:, :R], x[:, :R])


def small_store(rng, L=2, T=40, H=2, D=32):
    k = (rng.standard_normal((L, T, H, D)) * 2).astype(np.float32)
    v = (rng.standard_normal((L, T, H, D)) * 2).astype(np.float32)
    to_bits = lambda a: (torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))  # noqa: E731
    return to_bits(k), to_bits(v)


def test_inject_with_partial_rotation_and_e4m3_cache_images(oracle_mod):
    rng = np.random.default_rng(11)
    kb, vb = small_store(rng)
    lens = np.array([7, 9, 5, 11, 8], np.int32)
    offs = np.concatenate([[0], np.cumsum(lens)[:-1]]).astype(np.int64)
    table = np.array([3, 0, 5, 1, 2, 4], np.int32)
    ids = [3, 0, 4]
    plain = oracle_mod.inject(ids, offs, lens, kb, vb, 1e4, 5, table, 8, 6)
    part = oracle_mod.inject(ids, offs, lens, kb, vb, 1e4, 5, table, 8, 6, rotary_dim=16, k_scale=0.5, v_scale=0.25)
    assert part.m == plain.m and np.array_equal(part.slots, plain.slots) and np.array_equal(part.v, plain.v)
    # keys: tail copied exactly, leading block = rotation of a 16-dimensional head at the same positions
    src_tok = np.concatenate([np.arange(offs[f], offs[f] + lens[f]) for f in ids])
    x = oracle_mod.bf16_to_double(kb)[:, src_tok]  # [L, m, H, D]
    assert np.array_equal(part.k_ref[..., 16:], x[..., 16:])
    pos = 5 + np.arange(part.m)
    lead = oracle_mod.rope_rows(x[..., :16].reshape(-1, 16), np.tile(np.repeat(pos, 2), 2), 1e4)
    assert np.array_equal(part.k_ref[..., :16].reshape(-1, 16), lead)
    # quantised images decode to within half an e4m3 step (+ the bf16 rounding of the key) of value / scale
    for codes, ref, scale in ((part.k_fp8, oracle_mod.bf16_to_double(part.k_bf16), 0.5), (part.v_fp8, oracle_mod.bf16_to_double(part.v), 0.25)):
        target = ref / scale  # exact in binary32 for these two scales
        dec = oracle_mod.e4m3_to_double(codes)
        step = np.maximum(2.0 ** (np.floor(np.log2(np.maximum(np.abs(target), 2.0**-6))) - 3), 2.0**-9)
        assert np.all(np.abs(dec - np.clip(target, -448, 448)) <= step / 2)
        assert np.array_equal(codes, oracle_mod.e4m3_from_double(target.astype(np.float32).astype(np.float64)))
    # a value that e4m3 represents exactly survives quantisation with scale 1
    exact = np.array([[[[0.5, -1.75, 448.0, 2.0**-9] * 8]]], np.float32)  # [1, 1, 1, 32]
    eb = torch.from_numpy(exact).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    r = oracle_mod.inject([0], np.array([0], np.int64), np.array([1], np.int32), eb, eb, 1e4, 0, np.array([0], np.int32), 4, 1,
                          k_scale=1.0, v_scale=1.0)  # fmt: skip
    assert np.array_equal(oracle_mod.e4m3_to_double(r.v_fp8).reshape(-1), exact.reshape(-1).astype(np.float64))
    assert np.array_equal(oracle_mod.e4m3_to_double(r.k_fp8).reshape(-1), exact.reshape(-1).astype(np.float64))  # position 0: identity
