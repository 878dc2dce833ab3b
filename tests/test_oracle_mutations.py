"""Do the pins bite?  Each case plants one plausible mistake in a copy of the checker's C source (a dropped
term, a wrong sign or index, a transposed operand, a wrong constant), builds it, and demands that the pins
that do not depend on the checker itself notice: agreement with torch.nn.TransformerDecoderLayer in fp64,
incremental == full recompute, and the closed forms.  The mistakes live only in the temporary copy."""
import math
import os
import subprocess

import numpy as np
import pytest
import torch

from oracle import aed_oracle as orc
from paper_2503_05931_b200 import workloads as wl
from tests.helpers import torch_layer_logits

SRC = os.path.join(os.path.dirname(orc.__file__), "aed_oracle.c")

MUTATIONS = [
    ("8-bit format with one mantissa bit too many", "double quantum = ldexp(1.0, lead - 3);", "double quantum = ldexp(1.0, lead - 4);"),
    ("8-bit format with the wrong smallest normal exponent", "if (lead < -6) lead = -6;", "if (lead < -7) lead = -7;"),
    ("8-bit format saturating at the wrong value", "if (r > 448.0) r = 448.0;", "if (r > 480.0) r = 480.0;"),
    ("8-bit format rounding halves away from zero", "double r = nearbyint(a / quantum) * quantum;", "double r = floor(a / quantum + 0.5) * quantum;"),
    ("attention scale dropped", "real scale = (real)1 / (real)sqrt((double)dh);", "real scale = (real)1;"),
    ("softmax without max subtraction sign", "score[j] = (real)exp((double)(score[j] - mx));", "score[j] = (real)exp((double)(mx - score[j]));"),
    ("layernorm unbiased variance", "var /= (real)d;", "var /= (real)(d - 1);"),
    ("layernorm eps outside sqrt", "real inv = (real)1 / (real)sqrt((double)var + eps);", "real inv = (real)1 / ((real)sqrt((double)var) + (real)eps);"),
    ("embedding scale dropped", "double sq = sqrt((double)d);", "double sq = 1.0;"),
    ("sin and cos swapped", "double pe = (i % 2 == 0) ? sin(angle) : cos(angle);", "double pe = (i % 2 == 0) ? cos(angle) : sin(angle);"),
    ("position exponent uses i instead of the pair", "double angle = (double)t / pow(10000.0, (2.0 * pair) / (double)d);", "double angle = (double)t / pow(10000.0, (2.0 * i) / (double)d);"),
    ("key and value blocks swapped", "memcpy(Kl + (size_t)t * d, qkv + d, sizeof(real) * d);\n            memcpy(Vl + (size_t)t * d, qkv + 2 * d, sizeof(real) * d);",
     "memcpy(Kl + (size_t)t * d, qkv + 2 * d, sizeof(real) * d);\n            memcpy(Vl + (size_t)t * d, qkv + d, sizeof(real) * d);"),
    ("self-attention misses the current position", "attend(qkv, Kl, Vl, t + 1, H, dh, s,", "attend(qkv, Kl, Vl, t > 0 ? t : 1, H, dh, s,"),
    ("cross-attention residual dropped", "linear(w->w_o_c[l], BIAS(b_o_c, l), s, d, d, o);\n            for (int i = 0; i < d; ++i) x[i] += o[i];\n            /* feed-forward */",
     "linear(w->w_o_c[l], BIAS(b_o_c, l), s, d, d, o);\n            for (int i = 0; i < d; ++i) x[i] = o[i];\n            /* feed-forward */"),
    ("relu dropped", "for (int i = 0; i < F; ++i) if (hid[i] < 0) hid[i] = 0;", "for (int i = 0; i < F; ++i) if (hid[i] < -1e30) hid[i] = 0;"),
    ("ffn uses ln2 parameters", "orc_layernorm(x, w->ln3_g[l], w->ln3_b[l], d, cfg->ln_eps, a);\n            linear(w->w_ff1[l]", "orc_layernorm(x, w->ln2_g[l], w->ln2_b[l], d, cfg->ln_eps, a);\n            linear(w->w_ff1[l]"),
    ("weight matrix read transposed", "for (int i = 0; i < n_in; ++i) acc += (real)w[i] * x[i];\n        y[o] = acc;\n    }\n}\n\n/* same with a float input vector",
     "for (int i = 0; i < n_in; ++i) acc += (real)W[(size_t)i * n_out + o] * x[i];\n        y[o] = acc;\n    }\n}\n\n/* same with a float input vector"),
    ("heads read with the wrong stride", "for (int c = 0; c < dh; ++c) s += q[h * dh + c] * K[(size_t)j * d + h * dh + c];", "for (int c = 0; c < dh; ++c) s += q[h * dh + c] * K[(size_t)j * d + c * (d / dh) + h];"),
    ("argmax prefers the highest index on ties", "for (int i = 1; i < n; ++i) if (z[i] > z[best]) best = i;", "for (int i = 1; i < n; ++i) if (z[i] >= z[best]) best = i;"),
    ("cross values taken from the key block", "memcpy(Vc + (size_t)j * d, tmp + d, sizeof(real) * d);", "memcpy(Vc + (size_t)j * d, tmp, sizeof(real) * d);"),
    ("incremental decoder forgets the final layernorm bias", "orc_layernorm(x, w->final_ln_g, w->final_ln_b, d, cfg->ln_eps, a);\n        linear(w->w_out, w->b_out, a, V, d, z);\n        if (logits) for (int v = 0; v < V; ++v) logits[(size_t)t * V + v] = (double)z[v];\n        tok =",
     "orc_layernorm(x, w->final_ln_g, w->final_ln_g, d, cfg->ln_eps, a);\n        linear(w->w_out, w->b_out, a, V, d, z);\n        if (logits) for (int v = 0; v < V; ++v) logits[(size_t)t * V + v] = (double)z[v];\n        tok ="),
]


def _pins(precision):
    """The checker-independent pins on a small model; raises AssertionError if any fails."""
    model = dict(n_layers=2, d_model=32, n_heads=4, d_ffn=48, vocab=29, d_enc=32)
    w = wl.make_custom(model, [7], [6], seed=4, bias_std=0.3)
    rng = np.random.default_rng(9)
    d, NL = model["d_model"], model["n_layers"]
    for name in ("ln1", "ln2", "ln3"):
        w.weights[name + "_g"] = [rng.normal(1, 0.3, d).astype(np.float32) for _ in range(NL)]
        w.weights[name + "_b"] = [rng.normal(0, 0.3, d).astype(np.float32) for _ in range(NL)]
    w.weights["final_ln_g"] = rng.normal(1, 0.3, d).astype(np.float32)
    w.weights["final_ln_b"] = rng.normal(0, 0.3, d).astype(np.float32)
    for name in ("w_qkv", "w_o", "w_q_c", "w_kv_c", "w_o_c", "w_ff1", "w_ff2"):
        w.weights[name] = [(a * 8).astype(np.float32) for a in w.weights[name]]
    w.weights["w_out"][5] = w.weights["w_out"][17]          # a planted tie for the argmax rule
    m = orc.Model(w.model, w.weights)
    L = 6
    forced = rng.integers(0, model["vocab"], size=L)
    out = orc.decode(m, w.enc, L, forced=forced, precision=precision)
    full = orc.decode(m, w.enc, L, forced=forced, precision=precision, full_recompute=True)
    assert np.max(np.abs(out["logits"] - full["logits"])) <= 1e-12
    z = torch_layer_logits(model, w.weights, w.enc, forced)
    np.testing.assert_allclose(out["logits"], z, atol=1e-10)
    assert not np.any(out["next"] == 17)                    # ties go to the lowest index
    idx, _ = orc.argmax(np.array([1.0, 3.0, 3.0, 2.0]), precision=precision)
    assert idx == 1
    # 8-bit storage format of the cross-attention keys and values: nearest value of the format decoded from its bit
    # fields, ties to the even mantissa, saturation at the largest finite value
    vals = sorted({(m / 8.0 * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7))
                   for e in range(16) for m in range(8) if not (e == 15 and m == 7)})
    vals = np.array(vals)
    xs = np.concatenate([rng.normal(0, 1, 300), rng.normal(0, 0.01, 200), rng.uniform(200, 470, 50), [1e5, 0.1875 * 2.0 ** -6]])
    got = orc.round_e4m3(xs, precision=precision)
    for x, g in zip(xs, got):
        a = min(abs(x), 448.0)
        dist = np.abs(vals - a)
        near = vals[dist == dist.min()]
        assert abs(g) in near and (g < 0) == (x < 0 and g != 0), (x, g)
    mids = (vals[1:-1] + vals[2:]) / 2
    for lo, hi, g in zip(vals[1:-1], vals[2:], orc.round_e4m3(mids, precision=precision)):
        even = lo if int(round(lo / (2.0 ** -9 if lo < 2.0 ** -6 else 2.0 ** (math.floor(math.log2(lo)) - 3)))) % 2 == 0 else hi
        assert g == even, (lo, hi, g)


def test_pins_pass_on_the_real_checker():
    _pins("f64")


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(tmp_path, name, old, new):
    src = open(SRC).read()
    assert src.count(old) >= 1, f"snippet of '{name}' not found in the checker source"
    mutated = tmp_path / "mut.c"
    mutated.write_text(src.replace(old, new, 1))
    lib = tmp_path / "libmut.so"
    subprocess.run(["gcc", "-O1", "-std=c11", "-fPIC", "-shared", "-fopenmp", str(mutated), "-o", str(lib), "-lm"], check=True)
    tag = "mut_" + name
    orc.load_custom(tag, str(lib))
    with pytest.raises(AssertionError):
        _pins(tag)
