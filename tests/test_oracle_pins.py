"""Pins for the CPU checker: every check here is against something other than the checker itself
(invariants, closed forms, a library implementation of the same layer, the paper's parameter counts)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import aed_oracle as orc
from paper_2503_05931_b200 import workloads as wl
from tests.helpers import torch_layer_logits

SMALL = dict(n_layers=2, d_model=32, n_heads=4, d_ffn=64, vocab=50, d_enc=32)


def small_workload(seed=3, enc_lens=(5, 9, 3), dec_lens=(6, 4, 7), model=SMALL, **kw):
    return wl.make_custom(model, enc_lens, dec_lens, seed=seed, **kw)


def utt_enc(w, u):
    off = w.enc_offsets
    return w.enc[off[u]:off[u + 1]]


def pos_enc(t, d):
    pe = np.zeros(d)
    for i in range(0, d, 2):
        ang = t / (10000.0 ** (i / d))
        pe[i] = math.sin(ang)
        pe[i + 1] = math.cos(ang)
    return pe


# ----------------------------------------------------------------------------------------------
# P1: incremental KV-cache decoding equals brute-force full recompute of causal attention
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("forced", [False, True])
def test_incremental_equals_full_recompute(forced):
    w = small_workload()
    m = orc.Model(w.model, w.weights)
    rng = np.random.default_rng(0)
    for u in range(w.batch):
        L = int(w.dec_lens[u])
        f = rng.integers(0, w.model["vocab"], size=L) if forced else None
        a = orc.decode(m, utt_enc(w, u), L, forced=f)
        b = orc.decode(m, utt_enc(w, u), L, forced=f, full_recompute=True)
        assert np.max(np.abs(a["logits"] - b["logits"])) <= 1e-12
        assert np.array_equal(a["next"], b["next"])
        np.testing.assert_allclose(a["margin"], b["margin"], atol=1e-12)


def test_free_running_feeds_back_argmax():
    """Greedy run == teacher-forced run on [bos, next_0, next_1, ...]."""
    w = small_workload()
    m = orc.Model(w.model, w.weights)
    a = orc.decode(m, utt_enc(w, 0), 6, bos=1)
    forced = np.concatenate([[1], a["next"][:-1]])
    b = orc.decode(m, utt_enc(w, 0), 6, forced=forced)
    assert np.array_equal(a["logits"], b["logits"])


# ----------------------------------------------------------------------------------------------
# P2: batch-composition invariance
# ----------------------------------------------------------------------------------------------
def test_batch_composition_invariance():
    w = small_workload()
    m = orc.Model(w.model, w.weights)
    full = orc.decode_batch(m, w.enc, w.enc_lens, w.dec_lens, want_logits=True, n_threads=2)
    # alone
    for u in range(w.batch):
        alone = orc.decode(m, utt_enc(w, u), int(w.dec_lens[u]))
        assert np.array_equal(alone["logits"], full["logits"][u])
        assert np.array_equal(alone["next"], full["next"][u, :w.dec_lens[u]])
    # other order, other companions
    order = [2, 0]
    sub = w.subset(order)
    part = orc.decode_batch(m, sub.enc, sub.enc_lens, sub.dec_lens, want_logits=True, n_threads=1)
    for i, u in enumerate(order):
        assert np.array_equal(part["logits"][i], full["logits"][u])
    # garbage after the utterance's own frames in a padded buffer must not be read
    u = 1
    padded = np.concatenate([utt_enc(w, u), 1e6 * np.ones((7, w.model["d_enc"]), np.float32)])
    T = int(w.enc_lens[u])
    alone = orc.decode(m, padded[:T], int(w.dec_lens[u]))
    assert np.array_equal(alone["logits"], full["logits"][u])


# ----------------------------------------------------------------------------------------------
# P3: softmax rows sum to one, are non-negative, and are causal
# ----------------------------------------------------------------------------------------------
def test_softmax_rows_sum_to_one():
    w = small_workload()
    m = orc.Model(w.model, w.weights)
    L, T = 7, int(w.enc_lens[1])
    out = orc.decode(m, utt_enc(w, 1), L, trace=True)
    sp, cp = out["self_probs"], out["cross_probs"]
    assert sp.shape == (L, 2, 4, L) and cp.shape == (L, 2, 4, T)
    assert np.all(sp >= 0) and np.all(cp >= 0)
    np.testing.assert_allclose(cp.sum(-1), 1.0, atol=1e-12)
    np.testing.assert_allclose(sp.sum(-1), 1.0, atol=1e-12)
    for t in range(L):   # nothing from the future
        assert np.all(sp[t, :, :, t + 1:] == 0)
        assert np.all(sp[t, :, :, :t + 1] > 0)


# ----------------------------------------------------------------------------------------------
# P4: cross K/V carry no position => permuting encoder frames changes nothing
# ----------------------------------------------------------------------------------------------
def test_encoder_frame_permutation_invariance():
    w = small_workload()
    m = orc.Model(w.model, w.weights)
    enc = utt_enc(w, 1)
    perm = np.random.default_rng(5).permutation(enc.shape[0])
    a = orc.decode(m, enc, 5)
    b = orc.decode(m, enc[perm], 5)
    np.testing.assert_allclose(a["logits"], b["logits"], atol=1e-12)
    # ... while permuting the decoder inputs does change the result (positions matter there)
    f = np.array([1, 7, 9, 11, 13])
    c = orc.decode(m, enc, 5, forced=f)
    dd = orc.decode(m, enc, 5, forced=f[[0, 2, 1, 3, 4]])
    assert np.max(np.abs(c["logits"][-1] - dd["logits"][-1])) > 1e-6


# ----------------------------------------------------------------------------------------------
# P5: closed forms
# ----------------------------------------------------------------------------------------------
def test_layernorm_closed_forms():
    d = 64
    rng = np.random.default_rng(1)
    x = rng.normal(2.0, 3.0, size=d)
    y = orc.layernorm(x, np.ones(d), np.zeros(d), eps=1e-5)
    var = x.var()
    assert abs(y.mean()) < 1e-12
    assert abs(y.var() - var / (var + 1e-5)) < 1e-12
    g, b = rng.normal(size=d).astype(np.float32), rng.normal(size=d).astype(np.float32)
    yc = orc.layernorm(np.full(d, 4.25), g, b)
    np.testing.assert_allclose(yc, b.astype(np.float64), atol=1e-12)
    ref = torch.nn.functional.layer_norm(torch.tensor(x), (d,), torch.tensor(g, dtype=torch.float64),
                                         torch.tensor(b, dtype=torch.float64), 1e-5).numpy()
    np.testing.assert_allclose(orc.layernorm(x, g, b), ref, atol=1e-12)


def _zero(w, names):
    for n in names:
        w.weights[n] = [np.zeros_like(a) for a in w.weights[n]]


def test_zeroed_output_projections_reduce_to_one_matmul():
    """With every residual branch silenced the logits are LN(E[y] sqrt(d) + PE(t)) Wout^T."""
    w = small_workload()
    _zero(w, ["w_o", "b_o", "w_o_c", "b_o_c", "w_ff2", "b_ff2"])
    w.weights["final_ln_g"] = np.random.default_rng(2).normal(1, 0.1, SMALL["d_model"]).astype(np.float32)
    w.weights["final_ln_b"] = np.random.default_rng(3).normal(0, 0.1, SMALL["d_model"]).astype(np.float32)
    w.weights["b_out"] = np.random.default_rng(4).normal(0, 0.1, SMALL["vocab"]).astype(np.float32)
    m = orc.Model(w.model, w.weights)
    forced = np.array([1, 17, 4, 33])
    out = orc.decode(m, utt_enc(w, 0), 4, forced=forced)
    d = SMALL["d_model"]
    for t, y in enumerate(forced):
        x = w.weights["embed"][y].astype(np.float64) * math.sqrt(d) + pos_enc(t, d)
        xn = (x - x.mean()) / math.sqrt(x.var() + 1e-5)
        xn = xn * w.weights["final_ln_g"] + w.weights["final_ln_b"]
        z = w.weights["w_out"].astype(np.float64) @ xn + w.weights["b_out"]
        np.testing.assert_allclose(out["logits"][t], z, atol=1e-12)
        assert out["next"][t] == int(np.argmax(z))


def test_positional_encoding_values():
    """Embedding rows set to zero expose PE(t): PE(0) = (0,1,0,1,...), PE(t)[0:2] = (sin t, cos t)."""
    model = dict(SMALL, n_layers=1)
    w = wl.make_custom(model, [3], [4], seed=1)
    _zero(w, ["w_o", "b_o", "w_o_c", "b_o_c", "w_ff2", "b_ff2"])
    d, V = model["d_model"], model["vocab"]
    w.weights["embed"] = np.zeros((V, d), np.float32)
    # read out one coordinate of LN(PE) per vocabulary row
    w.weights["w_out"] = np.eye(V, d, dtype=np.float32)
    m = orc.Model(w.model, w.weights)
    out = orc.decode(m, w.enc, 4, forced=[1, 1, 1, 1])
    for t in range(4):
        pe = pos_enc(t, d)
        expect = (pe - pe.mean()) / math.sqrt(pe.var() + 1e-5)
        np.testing.assert_allclose(out["logits"][t, :d], expect, atol=1e-12)
    pe0 = np.tile([0.0, 1.0], d // 2)
    np.testing.assert_allclose(out["logits"][0, :d], (pe0 - 0.5) / math.sqrt(0.25 + 1e-5), atol=1e-12)
    # last pair rotates with wavelength 10000^((d-2)/d): nearly constant (0, 1) over 4 steps
    assert abs(pos_enc(3, d)[d - 2] - math.sin(3 / 10000 ** ((d - 2) / d))) < 1e-15


def _np_ln(x, g, b, eps=1e-5):
    return (x - x.mean()) / math.sqrt(x.var() + eps) * g + b


def test_single_frame_cross_attention_and_first_step_self_attention():
    """T = 1: the cross-attention output is Vc[0] whatever the query; t = 0: self-attention returns v_0.
    One layer, one step, so the whole decoder can be written out by hand."""
    model = dict(SMALL, n_layers=1)
    w = wl.make_custom(model, [1], [1], seed=9)
    W = {k: (v[0].astype(np.float64) if isinstance(v, list) else (None if v is None else v.astype(np.float64)))
         for k, v in w.weights.items()}
    d = model["d_model"]
    m = orc.Model(w.model, w.weights)
    out = orc.decode(m, w.enc, 1, forced=[1])
    x = W["embed"][1] * math.sqrt(d) + pos_enc(0, d)
    a = _np_ln(x, W["ln1_g"], W["ln1_b"])
    v0 = W["w_qkv"][2 * d:] @ a + W["b_qkv"][2 * d:]
    x = x + W["w_o"] @ v0 + W["b_o"]
    vc = W["w_kv_c"][d:] @ w.enc[0].astype(np.float64) + W["b_kv_c"][d:]
    x = x + W["w_o_c"] @ vc + W["b_o_c"]
    f = _np_ln(x, W["ln3_g"], W["ln3_b"])
    x = x + W["w_ff2"] @ np.maximum(W["w_ff1"] @ f + W["b_ff1"], 0) + W["b_ff2"]
    z = W["w_out"] @ _np_ln(x, W["final_ln_g"], W["final_ln_b"])
    np.testing.assert_allclose(out["logits"][0], z, atol=1e-12)


def test_zero_query_gives_uniform_attention():
    """Wq = bq = 0 (self and cross) makes every score 0, so each softmax row is uniform."""
    w = small_workload()
    d = SMALL["d_model"]
    for l in range(SMALL["n_layers"]):
        w.weights["w_qkv"][l][:d] = 0
        w.weights["b_qkv"][l][:d] = 0
        w.weights["w_q_c"][l][:] = 0
        w.weights["b_q_c"][l][:] = 0
    m = orc.Model(w.model, w.weights)
    T = int(w.enc_lens[0])
    out = orc.decode(m, utt_enc(w, 0), 5, trace=True)
    np.testing.assert_allclose(out["cross_probs"], 1.0 / T, atol=1e-15)
    for t in range(5):
        np.testing.assert_allclose(out["self_probs"][t, :, :, :t + 1], 1.0 / (t + 1), atol=1e-15)


# ----------------------------------------------------------------------------------------------
# P6: same layer as torch.nn.TransformerDecoderLayer(norm_first=True), fp64
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed", [0, 1])
def test_matches_torch_transformer_decoder_layer(seed):
    model = dict(n_layers=3, d_model=48, n_heads=6, d_ffn=80, vocab=37, d_enc=48)
    w = wl.make_custom(model, [11], [9], seed=seed, bias_std=0.3)
    rng = np.random.default_rng(seed + 100)
    d, NL = model["d_model"], model["n_layers"]
    # non-trivial LayerNorm parameters and larger weights so that every term matters
    for name in ("ln1", "ln2", "ln3"):
        w.weights[name + "_g"] = [rng.normal(1, 0.3, d).astype(np.float32) for _ in range(NL)]
        w.weights[name + "_b"] = [rng.normal(0, 0.3, d).astype(np.float32) for _ in range(NL)]
    w.weights["final_ln_g"] = rng.normal(1, 0.3, d).astype(np.float32)
    w.weights["final_ln_b"] = rng.normal(0, 0.3, d).astype(np.float32)
    w.weights["b_out"] = rng.normal(0, 0.3, model["vocab"]).astype(np.float32)
    for name in ("w_qkv", "w_o", "w_q_c", "w_kv_c", "w_o_c", "w_ff1", "w_ff2"):
        w.weights[name] = [(a * 8).astype(np.float32) for a in w.weights[name]]
    m = orc.Model(w.model, w.weights)
    L = 9
    forced = rng.integers(0, model["vocab"], size=L)
    out = orc.decode(m, w.enc, L, forced=forced)

    z = torch_layer_logits(model, w.weights, w.enc, forced)
    assert np.max(np.abs(z)) > 0.5          # the comparison is not vacuous
    np.testing.assert_allclose(out["logits"], z, atol=1e-10)
    assert np.array_equal(out["next"], z.argmax(-1))


# ----------------------------------------------------------------------------------------------
# P7: the paper's parameter arithmetic
# ----------------------------------------------------------------------------------------------
def test_layer_parameter_count_matches_paper():
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "param_counts.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                vals[k] = float(v)
    lo = (vals["canary_1b_methods"] - vals["small_decoder"]) / vals["decoder_layers_removed"]
    hi = (vals["canary_1b_table"] - vals["small_decoder"]) / vals["decoder_layers_removed"]
    per_layer = wl.layer_param_count(wl.MODELS["canary24"]) / 1e6
    assert lo - 0.05 <= per_layer <= hi + 0.05, (lo, per_layer, hi)
    d = 1024
    assert wl.layer_param_count(wl.MODELS["canary24"]) == 16 * d * d + 9 * d + 4096 + 6 * d


# ----------------------------------------------------------------------------------------------
# P8: determinism, and the fp32 build stays within the fp32-mode tolerance of the fp64 build
# ----------------------------------------------------------------------------------------------
def test_determinism_and_fp32_build():
    w = wl.make_workload("cfg1")
    m = orc.Model(w.model, w.weights)
    a = orc.decode_batch(m, w.enc, w.enc_lens, w.dec_lens, want_logits=True, n_threads=4)
    b = orc.decode_batch(m, w.enc, w.enc_lens, w.dec_lens, want_logits=True, n_threads=1)
    assert a["threads"] >= 1
    for x, y in zip(a["logits"], b["logits"]):
        assert np.array_equal(x, y)
    forced = np.full(a["next"].shape, 1, np.int32)
    forced[:, 1:] = np.where(a["next"][:, :-1] >= 0, a["next"][:, :-1], 0)
    c = orc.decode_batch(m, w.enc, w.enc_lens, w.dec_lens, forced=forced, want_logits=True, precision="f32")
    worst = max(np.max(np.abs(x - y)) for x, y in zip(a["logits"], c["logits"]))
    assert worst < 1e-4, worst


def test_workload_draws_are_seeded():
    a, b = wl.make_workload("cfg1"), wl.make_workload("cfg1")
    assert np.array_equal(a.enc, b.enc) and np.array_equal(a.weights["w_qkv"][1], b.weights["w_qkv"][1])
    assert a.batch == 4 and a.enc_lens.min() >= 20 and a.enc_lens.max() <= 60
    assert a.dec_lens.min() >= 8 and a.dec_lens.max() <= 32
    c = wl.make_workload("cfg2", with_weights=False, with_enc=False)
    assert c.batch == 64 and c.enc_lens.min() >= 13 and c.enc_lens.max() <= 500
    assert np.all(c.dec_lens >= 2) and np.all(c.dec_lens <= 240)
    r = wl.round_to_bf16(np.array([1.0, 1.00390625, 1.01171875, 3.14159], np.float32))
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.015625      # ties to even, both directions
    assert np.array_equal(wl.round_to_bf16(r), r)
    assert np.array_equal(r, torch.tensor([1.0, 1.00390625, 1.01171875, 3.14159]).bfloat16().float().numpy())


# ----------------------------------------------------------------------------------------------
# P9: argmax tie-break
# ----------------------------------------------------------------------------------------------
def test_argmax_lowest_index_on_ties():
    z = np.array([0.5, 2.0, -1.0, 2.0, 2.0, 1.5])
    idx, margin = orc.argmax(z)
    assert idx == 1 and margin == 0.0
    idx, margin = orc.argmax(np.array([0.0, -3.0, 4.0, 3.75]))
    assert idx == 2 and margin == 0.25
    # planted tie inside a full decode: two identical output rows
    w = small_workload()
    w.weights["w_out"][31] = w.weights["w_out"][12]
    m = orc.Model(w.model, w.weights)
    out = orc.decode(m, utt_enc(w, 0), 6)
    assert np.all(out["logits"][:, 31] == out["logits"][:, 12])
    assert not np.any(out["next"] == 31)


# ----------------------------------------------------------------------------------------------
# End-of-sequence rule: the token is emitted and counted, then the utterance stops.  Pinned against the
# run without the rule, which the pins above fix independently.
# ----------------------------------------------------------------------------------------------
def test_eos_run_is_the_free_run_cut_after_the_first_eos():
    w = small_workload(seed=12, enc_lens=(6, 4, 9, 5), dec_lens=(12, 12, 12, 12))
    m = orc.Model(w.model, w.weights)
    stopped_early = 0
    for u in range(w.batch):
        L = int(w.dec_lens[u])
        free = orc.decode(m, utt_enc(w, u), L)
        assert free["len"] == L and np.all(free["next"] >= 0)
        # every token the free run emits, as the end-of-sequence id: first step, a middle step, the last step
        for eos in sorted(set(int(t) for t in free["next"])):
            first = int(np.flatnonzero(free["next"] == eos)[0])
            cut = orc.decode(m, utt_enc(w, u), L, eos=eos)
            assert cut["len"] == first + 1
            assert np.array_equal(cut["next"][:first + 1], free["next"][:first + 1])
            assert np.all(cut["next"][first + 1:] == -1)
            assert np.array_equal(cut["logits"][:first + 1], free["logits"][:first + 1])
            assert np.all(cut["logits"][first + 1:] == 0.0)          # nothing is computed after the stop
            stopped_early += first + 1 < L
        assert orc.decode(m, utt_enc(w, u), L, eos=int(free["next"][0]))["len"] == 1          # planted at step 0
        last_only = [int(t) for i, t in enumerate(free["next"]) if i == L - 1 and t not in free["next"][:L - 1]]
        for eos in last_only:                                                                   # only at the last step
            assert orc.decode(m, utt_enc(w, u), L, eos=eos)["len"] == L
        absent = next(v for v in range(w.model["vocab"]) if v not in free["next"])
        same = orc.decode(m, utt_enc(w, u), L, eos=absent)
        assert same["len"] == L and np.array_equal(same["next"], free["next"])
    assert stopped_early > 0


def test_eos_in_a_batch_stops_each_utterance_on_its_own():
    w = small_workload(seed=12, enc_lens=(6, 4, 9, 5), dec_lens=(12, 7, 12, 3))
    m = orc.Model(w.model, w.weights)
    free = orc.decode_batch(m, w.enc, w.enc_lens, w.dec_lens)
    assert np.array_equal(free["lens"], w.dec_lens)
    eos = int(free["next"][0, 4])
    cut = orc.decode_batch(m, w.enc, w.enc_lens, w.dec_lens, eos=eos)
    for u in range(w.batch):
        L = int(w.dec_lens[u])
        hits = np.flatnonzero(free["next"][u, :L] == eos)
        expect = int(hits[0]) + 1 if len(hits) else L
        assert cut["lens"][u] == expect
        assert np.array_equal(cut["next"][u, :expect], free["next"][u, :expect])
        assert np.all(cut["next"][u, expect:] == -1)
    assert cut["lens"][0] <= 5


# ---- 8-bit storage of the cross-attention keys and values (an extension; the format is the OCP E4M3 one) ------------

def _e4m3_values():
    """Every finite value of the format, decoded from its bit fields: sign, 4 exponent bits (bias 7), 3 mantissa bits;
    exponent field 0 holds the subnormals; the code with all exponent and mantissa bits set is not a number."""
    vals = []
    for code in range(256):
        sign = -1.0 if code & 0x80 else 1.0
        e, m = (code >> 3) & 0xF, code & 0x7
        if e == 0xF and m == 0x7:
            continue
        vals.append(sign * (m / 8.0 * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7)))
    return np.array(sorted(set(vals)))


def test_e4m3_rounding_against_the_enumerated_format():
    vals = _e4m3_values()
    assert vals.max() == 448.0 and vals[vals > 0].min() == 2.0 ** -9 and len(vals) == 253
    # every value of the format is a fixed point
    assert np.array_equal(orc.round_e4m3(vals), vals)
    rng = np.random.default_rng(8)
    x = np.concatenate([rng.normal(0, 1, 4000), rng.normal(0, 100, 2000), rng.normal(0, 0.01, 2000),
                        rng.uniform(-2.0 ** -6, 2.0 ** -6, 1000), [449.0, 463.9, 464.0, 1e6, -1e6, 2.0 ** -10, 0.0]])
    got = orc.round_e4m3(x)
    clipped = np.clip(x, -448.0, 448.0)
    nearest = vals[np.argmin(np.abs(vals[None, :] - clipped[:, None]), axis=1)]
    dist = np.abs(vals[None, :] - clipped[:, None])
    best = dist.min(axis=1)
    ties = (np.isclose(dist, best[:, None], rtol=0, atol=0)).sum(axis=1) > 1
    assert np.array_equal(got[~ties], nearest[~ties])
    assert np.all(np.abs(got - clipped) <= best + 0.0)
    # ties go to the even mantissa: midpoints between neighbours
    pos = vals[vals > 0]
    mids = (pos[:-1] + pos[1:]) / 2
    r = orc.round_e4m3(mids)
    for lo, hi, v in zip(pos[:-1], pos[1:], r):
        assert v in (lo, hi)
        mant = v / 2.0 ** -9 if v < 2.0 ** -6 else (v / 2.0 ** np.floor(np.log2(v)) - 1.0) * 8
        assert int(round(mant)) % 2 == 0, (lo, hi, v)


def test_e4m3_rounding_against_torch():
    import torch
    if not hasattr(torch, "float8_e4m3fn"):
        pytest.skip("this torch has no float8_e4m3fn")
    rng = np.random.default_rng(9)
    x = np.concatenate([rng.normal(0, 1, 5000), rng.normal(0, 60, 3000), rng.uniform(-0.02, 0.02, 2000)])
    x = x[np.abs(x) < 440].astype(np.float32)                    # inside the finite range
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).to(torch.float32).numpy().astype(np.float64)
    assert np.array_equal(orc.round_e4m3(x.astype(np.float64)), want)


def test_cross_kv_in_e4m3_changes_what_it_should():
    """With the 8-bit store only the cross-attention keys and values change: a model whose cross-attention output
    projection is zero decodes identically, a normal one does not, and when the encoder states and weights make
    every key and value a value of the format already, nothing changes either."""
    model = dict(n_layers=2, d_model=128, n_heads=2, d_ffn=256, vocab=50, d_enc=64)
    w = wl.make_custom(model, [9, 4], [5, 5], dtype="fp32", seed=12, out_std=0.2)
    a = orc.decode_batch(orc.Model(w.model, w.weights), w.enc, w.enc_lens, w.dec_lens, want_logits=True)
    b = orc.decode_batch(orc.Model(w.model, w.weights, cross_kv_e4m3=True), w.enc, w.enc_lens, w.dec_lens, want_logits=True)
    diff = max(float(np.max(np.abs(x - y))) for x, y in zip(a["logits"], b["logits"]))
    assert 1e-6 < diff < 0.5
    w0 = dict(w.weights)
    w0["w_o_c"] = [np.zeros_like(m) for m in w.weights["w_o_c"]]
    w0["b_o_c"] = [np.zeros_like(m) for m in w.weights["b_o_c"]]
    a = orc.decode_batch(orc.Model(w.model, w0), w.enc, w.enc_lens, w.dec_lens, want_logits=True)
    b = orc.decode_batch(orc.Model(w.model, w0, cross_kv_e4m3=True), w.enc, w.enc_lens, w.dec_lens, want_logits=True)
    assert all(np.array_equal(x, y) for x, y in zip(a["logits"], b["logits"]))
    # keys and values that are small integers: one-hot encoder frames, integer weights, no bias
    w1 = dict(w.weights)
    rng = np.random.default_rng(4)
    w1["w_kv_c"] = [rng.integers(-8, 9, size=m.shape).astype(np.float32) for m in w.weights["w_kv_c"]]
    w1["b_kv_c"] = [np.zeros_like(m) for m in w.weights["b_kv_c"]]
    enc = np.zeros_like(w.enc)
    enc[np.arange(len(enc)), rng.integers(0, model["d_enc"], size=len(enc))] = 1.0
    a = orc.decode_batch(orc.Model(w.model, w1), enc, w.enc_lens, w.dec_lens, want_logits=True)
    b = orc.decode_batch(orc.Model(w.model, w1, cross_kv_e4m3=True), enc, w.enc_lens, w.dec_lens, want_logits=True)
    assert all(np.array_equal(x, y) for x, y in zip(a["logits"], b["logits"]))
