"""The 8-bit (E4M3) cross-attention K/V store against the CPU checker storing the same way.

Both sides round keys and values to the format after the projection (nearest, ties to even, saturating); everything
else is as in the bf16 configuration.  A key or value whose exact value lies within the GPU's accumulation error of a
rounding boundary can land on the other side of it, one step of the format (6 to 12 % of the element) apart, which is
why the logit tolerance here is derived separately (see TOL_E4M3)."""
import numpy as np
import pytest

from paper_2503_05931_b200 import workloads as wl
from tests.helpers import MARGIN, greedy_compare, oracle_reference, teacher_forced_compare

pytestmark = pytest.mark.gpu

MID = dict(n_layers=3, d_model=256, n_heads=4, d_ffn=512, vocab=1000, d_enc=192)
BIG = dict(n_layers=2, d_model=1024, n_heads=16, d_ffn=1024, vocab=2000, d_enc=1024)

# Tolerance on teacher-forced logits.  The tensor-core projection of an element (fp32 accumulation of bf16 products)
# differs from the checker's fp64 one by about 1e-3 relative; the format's steps are 2^-3 relative apart, so roughly
# one element in sixty rounds to the neighbouring value, an error of up to 2^-4 of that element.  In a 64-wide dot
# product that is one flipped element per score on average: the same order as the bf16 configuration's own error
# (K/V caches in bf16), and the measured maximum over the cases below stays under the bf16 tolerance.
TOL_E4M3 = 3e-2


def _run(w, rows, label, max_batch=None):
    from paper_2503_05931_b200 import binding
    ref = oracle_reference(w, rows, cross_kv_e4m3=True)
    plain = oracle_reference(w, rows)
    dec = binding.decoder_for_workload(w, cross_kv_e4m3=True, max_batch=max_batch)
    try:
        worst, compared, bad = teacher_forced_compare(dec, w, ref, rows)
        # how far the store moves the logits at all: the parity claim is only worth something if this is well above
        # the tolerance's noise floor
        moved = max(float(np.max(np.abs(a - b))) for a, b in zip(ref["logits"], plain["logits"]))
        print(f"[parity] e4m3 {label} B={w.batch}: max |logit diff| = {worst:.3e} over {compared} rows x steps "
              f"(the store itself moves the checker's logits by {moved:.3e})")
        assert compared > 0
        assert worst < TOL_E4M3
        assert not bad, f"argmax mismatches at margin > {MARGIN}: {bad[:5]}"
        n_tok, _ = greedy_compare(dec, w, ref, rows)
        print(f"[parity] e4m3 {label}: {n_tok} greedy tokens compared")
        assert n_tok > 0
    finally:
        dec.close()
    return worst, moved


def test_e4m3_store_ragged_multi_tile():
    enc_lens = [1, 63, 64, 65, 130, 257, 5, 200] + [17] * 62
    dec_lens = [1, 2, 70, 66, 5, 33, 64, 65] + [3] * 62
    w = wl.make_custom(MID, enc_lens, dec_lens, dtype="bf16", seed=21, out_std=0.1)
    _run(w, [0, 1, 2, 3, 4, 5, 6, 7, 8, 69], "ragged")


def test_e4m3_store_wide_model_and_bias():
    """d = 1024 (16 heads, four 256-feature tiles of the K/V projection per layer) with biases and LayerNorm parameters."""
    enc_lens = [300, 129, 128, 40, 7, 1] * 3
    dec_lens = [12, 9, 7, 5, 3, 2] * 3
    w = wl.make_custom(BIG, enc_lens, dec_lens, dtype="bf16", seed=23, out_std=0.1, ln_std=0.2, bias_std=0.1)
    worst, moved = _run(w, [0, 1, 2, 5, 17], "wide")
    assert moved > 3 * worst, "the 8-bit store should move the logits by clearly more than the parity error"


def test_e4m3_store_many_rows():
    """More than 128 rows: the path whose attention writes bf16 planes."""
    rng = np.random.default_rng(3)
    n = 150
    w = wl.make_custom(MID, rng.integers(1, 90, size=n), rng.integers(1, 6, size=n), dtype="bf16", seed=24, out_std=0.1)
    _run(w, [0, 1, 2, 70, 149], "150 rows")


def test_e4m3_store_through_slots():
    from paper_2503_05931_b200 import binding, streaming
    rng = np.random.default_rng(11)
    n, slots = 15, 4
    w = wl.make_custom(MID, rng.integers(1, 120, size=n), rng.integers(2, 20, size=n), dtype="bf16", seed=25, out_std=0.1)
    ref = oracle_reference(w, want_logits=False, cross_kv_e4m3=True)
    dec = binding.Decoder(w.model, w.weights, "bf16", max_batch=slots, max_total_enc_frames=slots * 120, max_enc_len=120,
                          max_dec_len=20, cross_kv_e4m3=True)
    try:
        out, _ = streaming.decode_stream(dec, dec.upload_encoder(w.enc), w.enc_lens, w.dec_lens, slots)
        compared = 0
        for u in range(n):
            assert len(out[u]) == int(w.dec_lens[u])
            for t in range(int(w.dec_lens[u])):
                if ref["margin"][u, t] <= MARGIN:
                    break
                assert out[u][t] == ref["next"][u, t], (u, t)
                compared += 1
        print(f"[parity] e4m3 slots: {compared} greedy tokens compared")
        assert compared > n
    finally:
        dec.close()


def test_e4m3_store_needs_bf16():
    from paper_2503_05931_b200 import binding
    w = wl.make_custom(MID, [5], [2], dtype="fp32", seed=1)
    with pytest.raises(binding.AedError) as e:
        binding.decoder_for_workload(w, cross_kv_e4m3=True)
    assert e.value.status == binding.AED_ERR_UNSUPPORTED
