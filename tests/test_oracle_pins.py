"""Pins for the CPU oracle: each part is checked against something other than itself -- closed
forms, invariants, a library AdamW, the paper's printed memory figures, brute force."""
import math
import os

import numpy as np
import pytest
import torch

import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                k, v = line.split()
                out[k] = float(v)
    return out


def paper_hp(**kw):
    g = read_golden("training_hparams.txt")
    hp = O.HParams(lr=g["lr"], beta1=g["beta1"], beta2=g["beta2"], eps=g["eps"],
                   weight_decay=g["weight_decay"], max_norm=g["max_grad_norm"], step=1)
    for k, v in kw.items():
        setattr(hp, k, v)
    return hp


def bf16_round(x):
    return O.bf16_bits_to_f32(O.f32_to_bf16_bits(np.asarray(x, np.float32)))


def make_tensor(rng, n, block, p_std=0.02, g_std=1e-3, bf16_param=False):
    p = rng.normal(0, p_std, n).astype(np.float32)
    g = O.f32_to_bf16_bits(rng.normal(0, g_std, n).astype(np.float32))
    if bf16_param:
        p = O.f32_to_bf16_bits(p)
    return O.OracleTensor(p, g, block)


# ---------------------------------------------------------------------------------------------
# P4: code tables
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("signed", [True, False])
def test_tables_structure(signed):
    T = O.code_table(signed)
    assert T.dtype == np.float32 and T.size == 256
    assert np.all(np.diff(T.astype(np.float64)) > 0), "strictly increasing"
    assert T[255] == 1.0 and 0.0 in T
    if signed:
        assert T[127] == 0.0
        # antisymmetric on 0..126 <-> 254..128, and no -1.0
        assert np.array_equal(T[:127], -T[254:127:-1])
        assert T[0] > -1.0
        mags = T[128:255].astype(np.float64)
        cells = [2 ** e for e in range(7)]
    else:
        assert T[0] == 0.0
        mags = T[1:255].astype(np.float64)
        cells = [2 ** (e + 1) for e in range(7)]
    # decade e holds `cells[e]` values inside (10^(e-7), 10^(e-6)), uniformly spaced by 0.9*d/cells
    pos = 0
    for e, n in enumerate(cells):
        d = 10.0 ** (e - 6)
        chunk = mags[pos: pos + n]
        assert np.all(chunk > 0.1 * d * (1 - 1e-6)) and np.all(chunk < d)
        if n > 1:
            np.testing.assert_allclose(np.diff(chunk), 0.9 * d / n, rtol=2e-5)
        # first value sits half a cell above the decade's lower edge
        np.testing.assert_allclose(chunk[0], d * (0.1 + 0.45 / n), rtol=1e-6)
        pos += n
    assert pos == mags.size


def test_table_named_values():
    qs, qu = O.code_table(True), O.code_table(False)
    # smallest magnitudes: one cell in the lowest signed decade -> 0.55e-6; two in the unsigned -> 0.325e-6
    assert qs[128] == np.float32(5.5e-7) and qs[126] == np.float32(-5.5e-7)
    assert qu[1] == np.float32(3.25e-7)
    # largest below one: 1 - 0.45/64 and 1 - 0.45/128
    assert qs[254] == np.float32(1 - 0.45 / 64) and qs[0] == np.float32(-(1 - 0.45 / 64))
    assert qu[254] == np.float32(1 - 0.45 / 128)


@pytest.mark.parametrize("signed", [True, False])
def test_round_trip_all_codes(signed):
    T = O.code_table(signed)
    for i in range(256):
        assert O.nearest(signed, T[i]) == i
        assert O.nearest_brute(signed, T[i]) == i


# ---------------------------------------------------------------------------------------------
# P5: nearest-code search == brute-force argmin
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("signed", [True, False])
def test_nearest_matches_brute_force(signed):
    rng = np.random.default_rng(5)
    T = O.code_table(signed)
    lo = -1.0 if signed else 0.0
    xs = [rng.uniform(lo, 1.0, 1000).astype(np.float32)]
    mag = np.exp(rng.uniform(math.log(1e-9), 0.0, 1000)).astype(np.float32)
    xs.append(mag * (rng.choice([-1.0, 1.0], 1000).astype(np.float32) if signed else np.float32(1.0)))
    mids = ((T[:-1].astype(np.float64) + T[1:].astype(np.float64)) / 2)
    m32 = mids.astype(np.float32)
    xs += [m32, np.nextafter(m32, np.float32(2)), np.nextafter(m32, np.float32(-2))]
    xs.append(np.array([lo, 0.0, 1.0, -0.0, 1e-30, 2.0, -2.0 if signed else 0.0], np.float32))
    for x in np.concatenate(xs):
        a, b = O.nearest(signed, x), O.nearest_brute(signed, x)
        assert a == b, (x, a, b)
        # and the result is a true nearest neighbour, lower index on ties
        d = np.abs(T.astype(np.float64) - np.float64(x))
        assert a == int(np.argmin(d))


def test_nearest_ties_go_low_and_clamp():
    T = O.code_table(False)
    # a mid-point that is exactly representable in fp32 must go to the lower index
    for k in range(1, 255):
        mid = (np.float64(T[k]) + np.float64(T[k + 1])) / 2
        if np.float64(np.float32(mid)) == mid:
            assert O.nearest(False, np.float32(mid)) == k
            break
    else:
        pytest.fail("no representable mid-point found")
    assert O.nearest(True, -1.0) == 0 and O.nearest(True, 1.0) == 255 and O.nearest(False, 1.0) == 255


# ---------------------------------------------------------------------------------------------
# P7: state layout vs the paper's printed optimizer-memory figures
# ---------------------------------------------------------------------------------------------
def test_state_bytes_match_paper_memory_rows():
    g = read_golden("gpt_oss_120b_state_memory.txt")
    N = g["trainable_params_billion"] * 1e9
    printed_diff = g["cpu_base_gib_hybrid_2pct"] - g["cpu_base_gib_full_8bit"]   # GiB
    frac_moved = 1.0 - g["eight_bit_fraction_hybrid"]     # share that goes fp32-state -> 8-bit
    block = int(g["block_size"])

    def per_param_8bit(block):
        n = 1 << 24
        code, scale = O.state_bytes(n, block)
        return 2.0 * (code + scale) / n       # two moments

    fp32_state = 8.0                           # two fp32 moments
    pred = frac_moved * N * (fp32_state - per_param_8bit(block)) / 2 ** 30
    # N is printed to 4 digits (+-0.005e9 params -> +-0.03 GiB); the GiB figures to 0.01
    assert abs(pred - printed_diff) < 0.05, (pred, printed_diff)
    # the same closed form with 2-byte codes or with no scales misses by far more than that
    assert abs(frac_moved * N * (fp32_state - 4.0) / 2 ** 30 - printed_diff) > 100
    # ragged sizes: one scale per started block
    assert O.state_bytes(4097, 4096) == (4097, 8) and O.state_bytes(0, 4096) == (0, 0)
    assert O.state_bytes(4096, 4096) == (4096, 4)


# ---------------------------------------------------------------------------------------------
# P3: norm and clip factor
# ---------------------------------------------------------------------------------------------
def test_norm_of_ones_and_clip_factor():
    n = 1 << 20
    t = O.OracleTensor(np.zeros(n, np.float32), O.f32_to_bf16_bits(np.ones(n, np.float32)), 2048)
    S = O.sqnorm([t])
    assert S == float(n)                     # exact: ||g|| = sqrt(N)
    c, nf = O.clip_factor(S, 1.0)
    assert not nf and c == np.float32(1.0 / (math.sqrt(n) + 1e-6))
    c, _ = O.clip_factor(S, 1e9)
    assert c == 1.0                          # min(1, .)
    for off in (0.0, -1.0, float("inf")):    # clipping disabled
        assert O.clip_factor(S, off) == (1.0, False)
    for bad in (float("nan"), float("inf")):
        assert O.clip_factor(bad, 1.0)[1] is True
    # accumulates across calls / chunks and over dtypes
    t2 = O.OracleTensor(np.zeros(3, np.float32), np.array([3.0, 4.0, 0.0], np.float32), 2048)
    assert O.sqnorm([t2], 7.0) == 32.0
    assert O.sqnorm([t, t2]) == float(n) + 25.0


def test_norm_against_numpy_fp64():
    rng = np.random.default_rng(11)
    ts = [make_tensor(rng, n, 2048) for n in (1, 7, 2048, 5000, 100_003)]
    ref = sum(float(np.sum(O.bf16_bits_to_f32(t.grad).astype(np.float64) ** 2)) for t in ts)
    assert abs(O.sqnorm(ts) - ref) <= 1e-12 * ref


def test_clipped_update_is_scale_invariant():
    # with the clip active, c*g is (almost) independent of the gradient's scale
    rng = np.random.default_rng(3)
    n = 4096
    g = rng.normal(0, 1, n).astype(np.float32)
    outs = []
    for k in (1.0, 64.0):
        gb = O.f32_to_bf16_bits(bf16_round(g) * np.float32(k))     # power-of-two scale keeps bf16 exact
        t = O.OracleTensor(np.zeros(n, np.float32), gb, 2048)
        S = O.sqnorm([t])
        c, _ = O.clip_factor(S, 1.0)
        outs.append(np.float64(c) * O.bf16_bits_to_f32(gb).astype(np.float64))
        assert abs(np.linalg.norm(outs[-1]) - 1.0) < 1e-5          # clipped norm == max_norm
    np.testing.assert_allclose(outs[0], outs[1], rtol=1e-6)


# ---------------------------------------------------------------------------------------------
# P1 / P2: Adam arithmetic (quantization disabled) against closed forms and torch.optim.AdamW
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("betas", [(0.9, 0.999), (0.5, 0.75), (0.0, 0.0)])
def test_first_step_closed_form(betas):
    rng = np.random.default_rng(1)
    n = 1000
    p0 = rng.normal(0, 0.02, n).astype(np.float32)
    g = rng.normal(0, 1e-3, n).astype(np.float32)
    g[:10] = 0.0
    hp = paper_hp(beta1=betas[0], beta2=betas[1], step=1)
    p = p0.copy(); m = np.zeros(n, np.float32); v = np.zeros(n, np.float32)
    O.step_fp32state(p, g.copy(), m, v, hp, 1.0)
    lr, wd, eps = np.float64(np.float32(hp.lr)), np.float64(np.float32(hp.weight_decay)), np.float64(np.float32(hp.eps))
    g64, p64 = g.astype(np.float64), p0.astype(np.float64)
    # bias-corrected first step: m_hat = g, v_hat = g^2 for ANY betas
    ref = p64 * (1 - lr * wd) - lr * g64 / (np.abs(g64) + eps)
    np.testing.assert_allclose(p, ref, rtol=2e-6, atol=1e-9)
    # zero gradient: pure decoupled decay, exactly one fp32 multiply
    assert np.array_equal(p[:10], p0[:10] * np.float32(1 - lr * wd))
    assert np.all(m[:10] == 0) and np.all(v[:10] == 0)


def test_eight_bit_first_step_matches_closed_form():
    rng = np.random.default_rng(2)
    n = 5000
    t = make_tensor(rng, n, 2048)
    p0 = t.param.copy()
    g64 = O.bf16_bits_to_f32(t.grad).astype(np.float64)
    hp = paper_hp(max_norm=0.0)
    assert O.hybrid8_step([t], 2048, hp, O.sqnorm([t])) == 0
    ref = p0.astype(np.float64) * (1 - 1e-5 * 0.01) - 1e-5 * g64 / (np.abs(g64) + 1e-8)
    np.testing.assert_allclose(t.param, ref, rtol=3e-6, atol=1e-9)


def test_fp32_state_mode_matches_torch_adamw():
    torch.manual_seed(0)
    n, steps = 257, 6
    hp = paper_hp(lr=1e-3, weight_decay=0.1)
    p_t = torch.nn.Parameter(torch.randn(n) * 0.02)
    # the oracle's hyper-parameters are fp32 fields; hand the library the same (fp32-representable) values
    f32 = lambda x: float(np.float32(x))  # noqa: E731
    opt = torch.optim.AdamW([p_t], lr=f32(hp.lr), betas=(f32(hp.beta1), f32(hp.beta2)), eps=f32(hp.eps),
                            weight_decay=f32(hp.weight_decay), foreach=False, fused=False)
    p = p_t.detach().numpy().copy(); m = np.zeros(n, np.float32); v = np.zeros(n, np.float32)
    for k in range(1, steps + 1):
        g = (torch.randn(n) * (1e-2 if k % 2 else 1.0)).float()
        p_t.grad = g.clone()
        opt.step()
        hp.step = k
        O.step_fp32state(p, g.numpy().copy(), m, v, hp, 1.0)
        np.testing.assert_allclose(p, p_t.detach().numpy(), rtol=1e-6, atol=1e-9)
        st = opt.state[p_t]
        # the library forms m with lerp (m + (1-b1)(g-m)): same value, other rounding order
        np.testing.assert_allclose(m, st["exp_avg"].numpy(), rtol=1e-6, atol=3e-7 * float(np.abs(m).max()))
        np.testing.assert_allclose(v, st["exp_avg_sq"].numpy(), rtol=1e-6, atol=1e-15)


def test_fp32_state_mode_matches_fp64_recurrence_with_clip():
    rng = np.random.default_rng(4)
    n = 300
    hp = paper_hp()
    p = rng.normal(0, 0.02, n).astype(np.float32); m = np.zeros(n, np.float32); v = np.zeros(n, np.float32)
    P, M, V = p.astype(np.float64), np.zeros(n), np.zeros(n)
    b1, b2 = np.float64(np.float32(0.9)), np.float64(np.float32(0.999))
    lr, wd, eps = (np.float64(np.float32(x)) for x in (hp.lr, hp.weight_decay, hp.eps))
    for k in range(1, 5):
        g = rng.normal(0, 1e-3, n).astype(np.float32)
        c = 0.25 * k
        hp.step = k
        O.step_fp32state(p, g.copy(), m, v, hp, c)
        G = np.float64(np.float32(c)) * g.astype(np.float64)
        M = b1 * M + (1 - b1) * G
        V = b2 * V + (1 - b2) * G * G
        P = P * (1 - lr * wd) - lr / (1 - b1 ** k) * M / (np.sqrt(V / (1 - b2 ** k)) + eps)
        np.testing.assert_allclose(p, P, rtol=2e-6, atol=1e-9)


def test_step_scalars():
    hp = paper_hp(step=3)
    s = O.step_scalars(hp)
    b1, b2 = np.float64(np.float32(0.9)), np.float64(np.float32(0.999))
    assert s["step_size"] == np.float32(np.float64(np.float32(1e-5)) / (1 - b1 ** 3))
    assert s["inv_sqrt_bc2"] == np.float32(1 / math.sqrt(1 - b2 ** 3))
    assert s["omb1"] == np.float32(1 - b1) and s["omb2"] == np.float32(1 - b2)
    assert s["decay"] == np.float32(1 - np.float64(np.float32(1e-5)) * np.float64(np.float32(0.01)))


# ---------------------------------------------------------------------------------------------
# P6: block-wise absmax / requantization invariants
# ---------------------------------------------------------------------------------------------
def code_gap_halfwidth(T, code):
    """Half the distance from T[code] to its farther neighbour (the cell's worst-case error)."""
    T = T.astype(np.float64)
    left = np.where(code > 0, T[code] - T[np.maximum(code - 1, 0)], 0.0)
    right = np.where(code < 255, T[np.minimum(code + 1, 255)] - T[code], 0.0)
    return np.maximum(left, right) / 2


@pytest.mark.parametrize("block", [2048, 4096])
@pytest.mark.parametrize("bf16_param", [False, True])
def test_requant_invariants(block, bf16_param):
    rng = np.random.default_rng(6)
    n = 3 * block + 777
    t = make_tensor(rng, n, block, bf16_param=bf16_param)
    QS, QU = O.code_table(True), O.code_table(False)
    hp = paper_hp(max_norm=0.0)
    b1, b2 = np.float32(hp.beta1), np.float32(hp.beta2)
    omb1, omb2 = np.float32(1 - np.float64(b1)), np.float32(1 - np.float64(b2))
    for k in range(1, 4):
        t.set_grad(O.f32_to_bf16_bits(rng.standard_t(3, n).astype(np.float32) * np.float32(1e-3)))
        m_old = O.dequant(True, t.m_code, t.m_absmax, block)
        v_old = O.dequant(False, t.v_code, t.v_absmax, block)
        hp.step = k
        O.hybrid8_step([t], block, hp, O.sqnorm([t]))
        g = O.bf16_bits_to_f32(t.grad)
        m2 = b1 * m_old + omb1 * g                 # fp32 numpy ops, one rounding each
        v2 = b2 * v_old + omb2 * (g * g)
        blk = np.arange(n) // block
        nb = (n + block - 1) // block
        am = np.array([np.max(np.abs(m2[blk == b])) for b in range(nb)], np.float32)
        av = np.array([np.max(v2[blk == b]) for b in range(nb)], np.float32)
        assert np.array_equal(t.m_absmax, am) and np.array_equal(t.v_absmax, av)   # scale == block max, exactly
        for b in range(nb):
            idx = np.where(blk == b)[0]
            i = idx[np.argmax(np.abs(m2[idx]))]
            assert t.m_code[i] == (255 if m2[i] > 0 else 0)
            assert t.v_code[idx[np.argmax(v2[idx])]] == 255
        # per-element reconstruction error: at most half the local code gap (in units of the scale)
        m_new = O.dequant(True, t.m_code, t.m_absmax, block).astype(np.float64)
        v_new = O.dequant(False, t.v_code, t.v_absmax, block).astype(np.float64)
        tol_m = am[blk].astype(np.float64) * (code_gap_halfwidth(QS, t.m_code) + 2e-7)
        tol_v = av[blk].astype(np.float64) * (code_gap_halfwidth(QU, t.v_code) + 2e-7)
        # code 0 of the signed map also absorbs everything below it (there is no -1.0)
        tol_m = np.where(t.m_code == 0, am[blk] * (1.0 - 0.99296874) * 1.0001, tol_m)
        assert np.all(np.abs(m_new - m2) <= tol_m)
        assert np.all(np.abs(v_new - v2) <= tol_v)
        # codes are monotone in the value inside a block
        idx = np.where(blk == 1)[0]
        assert np.all(np.diff(t.m_code[idx][np.argsort(m2[idx], kind="stable")].astype(int)) >= 0)
        assert np.all(np.diff(t.v_code[idx][np.argsort(v2[idx], kind="stable")].astype(int)) >= 0)


def test_zero_block_gives_zero_codes_and_scale():
    n, block = 2 * 2048 + 5, 2048
    p = np.full(n, 0.5, np.float32)
    t = O.OracleTensor(p.copy(), np.zeros(n, np.uint16), block)
    t.m_code[:] = 7; t.v_code[:] = 9          # byte garbage with zero scales decodes to zero (A7)
    hp = paper_hp()
    O.hybrid8_step([t], block, hp, 0.0)
    assert np.all(t.m_code == 127) and np.all(t.v_code == 0)
    assert np.all(t.m_absmax == 0) and np.all(t.v_absmax == 0)
    assert np.array_equal(t.param, p * np.float32(1 - 1e-5 * 0.01))     # decay still applied


def test_byte_zero_state_equals_value_zero_state():
    rng = np.random.default_rng(8)
    a = make_tensor(rng, 5000, 2048)
    b = O.OracleTensor(a.param.copy(), a.grad.copy(), 2048, m_code=np.zeros(5000, np.uint8),
                       v_code=np.zeros(5000, np.uint8))
    hp = paper_hp()
    S = O.sqnorm([a])
    O.hybrid8_step([a], 2048, hp, S); O.hybrid8_step([b], 2048, hp, S)
    for k in ("param", "m_code", "v_code", "m_absmax", "v_absmax"):
        assert np.array_equal(getattr(a, k), getattr(b, k))


def test_state_init_values():
    t = O.OracleTensor(np.zeros(5000, np.float32), np.zeros(5000, np.uint16), 2048,
                       m_code=np.full(5000, 3, np.uint8), v_code=np.full(5000, 3, np.uint8),
                       m_absmax=np.ones(3, np.float32), v_absmax=np.ones(3, np.float32))
    O.state_init([t], 2048)
    assert np.all(t.m_code == 127) and np.all(t.v_code == 0)
    assert np.all(t.m_absmax == 0) and np.all(t.v_absmax == 0)
    assert np.all(O.dequant(True, t.m_code, np.ones(3, np.float32), 2048) == 0)


# ---------------------------------------------------------------------------------------------
# P8: zero-gradient behaviour of the codes
# ---------------------------------------------------------------------------------------------
def test_zero_gradient_code_invariance():
    rng = np.random.default_rng(9)
    block, nb = 2048, 40
    n = nb * block
    t = make_tensor(rng, n, block, g_std=1e-3)
    hp = paper_hp(max_norm=0.0)
    for k in (1, 2):
        t.set_grad(O.f32_to_bf16_bits(rng.normal(0, 1e-3, n).astype(np.float32)))
        hp.step = k
        O.hybrid8_step([t], block, hp, 1.0)
    mc, vc = t.m_code.copy(), t.v_code.copy()
    t.set_grad(np.zeros(n, np.uint16))
    hp.step = 3
    O.hybrid8_step([t], block, hp, 0.0)
    assert np.array_equal(t.v_code, vc)        # v codes invariant in every block
    seen_neg = seen_pos = False
    for b in range(nb):
        sl = slice(b * block, (b + 1) * block)
        if (mc[sl] == 255).any():              # block max was positive: sits on +1.0, codes invariant
            assert np.array_equal(t.m_code[sl], mc[sl]); seen_pos = True
        else:                                  # block max was negative: sits on code 0 (no -1.0);
            seen_neg = True                    # the scale shrinks by |QS[0]| and only 254 -> 255 may move
            diff = np.where(t.m_code[sl] != mc[sl])[0]
            assert np.all(mc[sl][diff] == 254) and np.all(t.m_code[sl][diff] == 255)
    assert seen_neg and seen_pos


# ---------------------------------------------------------------------------------------------
# P9 / P10: chunk invariance, skip on non-finite
# ---------------------------------------------------------------------------------------------
def clone(ts):
    return [O.OracleTensor(t.param.copy(), t.grad.copy(), t.block, t.m_code.copy(), t.v_code.copy(),
                           t.m_absmax.copy(), t.v_absmax.copy()) for t in ts]


def same(a, b):
    return all(np.array_equal(getattr(x, k), getattr(y, k)) for x, y in zip(a, b)
               for k in ("param", "m_code", "v_code", "m_absmax", "v_absmax"))


def test_chunk_invariance():
    rng = np.random.default_rng(10)
    ts = [make_tensor(rng, n, 2048) for n in (1, 2047, 2048, 2049, 10_000, 333)]
    hp = paper_hp()
    a, b = clone(ts), clone(ts)
    S = O.sqnorm(a)
    O.hybrid8_step(a, 2048, hp, S)
    for chunk in (b[:2], b[2:3], b[3:]):
        O.hybrid8_step(chunk, 2048, hp, S)
    assert same(a, b)
    assert not same(a, ts)


def test_nonfinite_norm_skips_everything():
    rng = np.random.default_rng(12)
    ts = [make_tensor(rng, n, 2048) for n in (100, 5000)]
    for bad in (0x7FC0, 0x7F80, 0xFF80):       # NaN, +Inf, -Inf as bf16 bits
        a = clone(ts)
        a[1].grad[4321] = bad
        before = clone(a)
        S = O.sqnorm(a)
        assert not math.isfinite(S)
        assert O.hybrid8_step(a, 2048, paper_hp(), S) & 1
        assert same(a, before)
    a = clone(ts)
    assert O.hybrid8_step(a, 2048, paper_hp(), O.sqnorm(a)) == 0


# ---------------------------------------------------------------------------------------------
# whole step: definitional brute-force variant, bf16 rounding, and distance from the fp32 trajectory
# ---------------------------------------------------------------------------------------------
def test_search_step_equals_brute_force_step():
    rng = np.random.default_rng(13)
    ts = [make_tensor(rng, n, 2048) for n in (2048 * 3 + 100, 900)]
    a, b = clone(ts), clone(ts)
    hp = paper_hp()
    for k in (1, 2, 3):
        for x in (a, b):
            for t, u in zip(x, ts):
                t.set_grad(u.grad if k == 1 else np.roll(u.grad, k))
        hp.step = k
        S = O.sqnorm(a)
        O.hybrid8_step(a, 2048, hp, S, brute=False)
        O.hybrid8_step(b, 2048, hp, S, brute=True)
        assert same(a, b)


def test_bf16_param_is_rne_of_fp32_result():
    rng = np.random.default_rng(14)
    n = 6000
    p = bf16_round(rng.normal(0, 0.02, n).astype(np.float32))
    g = O.f32_to_bf16_bits(rng.normal(0, 1e-3, n).astype(np.float32))
    a = O.OracleTensor(p.copy(), g, 2048)
    b = O.OracleTensor(O.f32_to_bf16_bits(p), g, 2048)
    hp = paper_hp(lr=1e-2)
    S = O.sqnorm([a])
    O.hybrid8_step([a], 2048, hp, S); O.hybrid8_step([b], 2048, hp, S)
    assert np.array_equal(O.f32_to_bf16_bits(a.param), b.param)
    assert np.array_equal(a.m_code, b.m_code) and np.array_equal(a.v_code, b.v_code)
    # RNE helper itself: halfway cases go to even
    assert O.f32_to_bf16_bits(np.array([1.00390625], np.float32))[0] == 0x3F80      # 1 + 2^-8 -> 1.0
    assert O.f32_to_bf16_bits(np.array([1.01171875], np.float32))[0] == 0x3F82      # 1 + 3*2^-8 -> 1 + 2^-6


def test_quantized_trajectory_stays_near_fp32_trajectory():
    rng = np.random.default_rng(15)
    n, block = 4 * 2048, 2048
    p0 = rng.normal(0, 0.02, n).astype(np.float32)
    t = O.OracleTensor(p0.copy(), np.zeros(n, np.uint16), block)
    p = p0.copy(); m = np.zeros(n, np.float32); v = np.zeros(n, np.float32)
    hp = paper_hp(max_norm=0.0)
    for k in (1, 2, 3):
        g = O.f32_to_bf16_bits(rng.normal(0, 1e-3, n).astype(np.float32))
        t.set_grad(g); hp.step = k
        O.hybrid8_step([t], block, hp, 1.0)
        O.step_fp32state(p, O.bf16_bits_to_f32(g), m, v, hp, 1.0)
        mq = O.dequant(True, t.m_code, t.m_absmax, block)
        vq = O.dequant(False, t.v_code, t.v_absmax, block)
        # moments: within a few code gaps (<= ~1.5 % of the block scale per step, accumulated)
        assert np.max(np.abs(mq - m)) <= 0.03 * k * np.max(np.abs(m))
        assert np.max(np.abs(vq - v)) <= 0.03 * k * np.max(v)
        # every parameter moved by at most ~lr per step in both, so they stay within 2*k*lr
        assert np.max(np.abs(t.param - p)) <= 2 * k * 1e-5


# ---------------------------------------------------------------------------------------------
# hybrid split: tensors with plain fp32 moments inside the same step
# ---------------------------------------------------------------------------------------------
def test_fp32_state_tensors_in_the_step_equal_the_pinned_fp32_mode():
    rng = np.random.default_rng(21)
    n = 3000
    p0 = rng.normal(0, 0.02, n).astype(np.float32)
    t32 = O.OracleTensor(p0.copy(), np.zeros(n, np.uint16), 4096, fp32_state=True)
    t8 = O.OracleTensor(p0.copy(), np.zeros(n, np.uint16), 4096)
    tb = O.OracleTensor(O.f32_to_bf16_bits(p0), np.zeros(n, np.uint16), 4096, fp32_state=True)
    p = p0.copy(); m = np.zeros(n, np.float32); v = np.zeros(n, np.float32)
    pb = bf16_round(p0); mb = np.zeros(n, np.float32); vb = np.zeros(n, np.float32)
    hp = paper_hp(max_norm=0.5)
    for k in (1, 2, 3):
        g = O.f32_to_bf16_bits(rng.normal(0, 1e-3, n).astype(np.float32))
        for t in (t32, t8, tb):
            t.set_grad(g)
        S = O.sqnorm([t32, t8])
        c, _ = O.clip_factor(S, hp.max_norm)
        hp.step = k
        assert O.hybrid8_step([t32, t8, tb], 4096, hp, S) == 0       # mixed list, one clip factor
        O.step_fp32state(p, O.bf16_bits_to_f32(g), m, v, hp, c)      # the mode pinned against torch.optim.AdamW
        assert np.array_equal(t32.param, p) and np.array_equal(t32.m_code, m) and np.array_equal(t32.v_code, v)
        # bf16 parameters: same moments, parameter = RNE of the fp32 result computed from the bf16 parameter
        O.step_fp32state(pb, O.bf16_bits_to_f32(g), mb, vb, hp, c)
        assert np.array_equal(tb.param, O.f32_to_bf16_bits(pb))
        pb = bf16_round(pb)
        assert np.array_equal(tb.m_code, m)
    assert t8.m_code.dtype == np.uint8 and not np.array_equal(t8.param, p0)
    z = O.OracleTensor(p0.copy(), np.zeros(n, np.uint16), 4096, m_code=np.ones(n, np.float32), v_code=np.ones(n, np.float32))
    O.state_init([z], 4096)
    assert not z.m_code.any() and not z.v_code.any()


def test_oracle_is_clean_under_address_and_ub_sanitizers(tmp_path):
    """The oracle compiled with AddressSanitizer and UndefinedBehaviorSanitizer runs its whole path (state init,
    norm, steps with both quantizers, skip) over exactly-sized heap arrays of awkward lengths without a report."""
    import shutil
    import subprocess
    if shutil.which("g++") is None:
        pytest.skip("no g++")
    here = os.path.dirname(os.path.abspath(__file__))
    exe = str(tmp_path / "oracle_sanitized")
    cmd = ["g++", "-O1", "-g", "-std=c++17", "-ffp-contract=off", "-fsanitize=address,undefined",
           "-fno-sanitize-recover=all", "-o", exe, os.path.join(here, "oracle_sanitizer_driver.cpp")]
    built = subprocess.run(cmd, capture_output=True, text=True)
    if built.returncode != 0 and "sanitize" in (built.stderr or "") and "cannot find" in built.stderr:
        pytest.skip("sanitizer runtime not installed")
    assert built.returncode == 0, built.stderr[-2000:]
    run = subprocess.run([exe], capture_output=True, text=True, timeout=300,
                         env=dict(os.environ, ASAN_OPTIONS="detect_leaks=1", UBSAN_OPTIONS="print_stacktrace=1"))
    assert run.returncode == 0, (run.stdout + run.stderr)[-3000:]
    assert "sanitizer run clean" in run.stdout
