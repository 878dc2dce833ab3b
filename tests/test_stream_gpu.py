"""Continuous batching (slots that utterances enter and leave one by one) against the CPU checker: an utterance's
greedy tokens do not depend on what else is in the batch, so every utterance of the stream must come out as the
checker decodes it alone, whatever slot it went through and whoever used that slot before."""
import numpy as np
import pytest

from paper_2503_05931_b200 import workloads as wl
from tests.helpers import MARGIN, oracle_reference

pytestmark = pytest.mark.gpu

MID = dict(n_layers=3, d_model=256, n_heads=4, d_ffn=512, vocab=1000, d_enc=192)


def _stream(dtype, n, seed, eos=-1):
    rng = np.random.default_rng(seed)
    enc_lens = rng.integers(1, 150, size=n)
    enc_lens[:3] = [150, 1, 129]
    dec_lens = rng.integers(1, 40, size=n)
    dec_lens[:4] = [40, 1, 2, 33]
    w = wl.make_custom(MID, enc_lens, dec_lens, dtype=dtype, seed=seed, out_std=0.1, ln_std=0.2)
    ref = oracle_reference(w, want_logits=False, eos=eos)
    return w, ref


def _check_against_checker(w, ref, out, lens_expected):
    compared = 0
    for u in range(w.batch):
        L = int(lens_expected[u])
        assert len(out[u]) == L, (u, len(out[u]), L)
        for t in range(L):
            if ref["margin"][u, t] <= MARGIN:
                break
            assert out[u][t] == ref["next"][u, t], f"utterance {u} step {t}: {out[u][t]} vs {ref['next'][u, t]}"
            compared += 1
    return compared


@pytest.mark.parametrize("dtype,slots", [("fp32", 5), ("bf16", 5), ("bf16", 1), ("bf16", 24)])
def test_stream_through_slots_matches_the_checker(dtype, slots):
    from paper_2503_05931_b200 import binding, streaming
    n = 23
    w, ref = _stream(dtype, n, seed=31 + slots)
    dec = binding.Decoder(w.model, w.weights, dtype, max_batch=max(slots, 2), max_total_enc_frames=slots * 150,
                          max_enc_len=150, max_dec_len=40)
    try:
        enc = dec.upload_encoder(w.enc)
        order = np.random.default_rng(5).permutation(n)
        out, stats = streaming.decode_stream(dec, enc, w.enc_lens, w.dec_lens, slots, order=order)
        compared = _check_against_checker(w, ref, out, w.dec_lens)
        print(f"[parity] stream {dtype} slots={slots}: {compared} greedy tokens compared, {stats}")
        assert compared > n
        # every step the host issued had at least one decoding row, and no row ran past its forced length
        assert stats["row_steps"] == int(w.dec_lens.sum())
        if slots == 1:
            assert stats["steps"] == int(w.dec_lens.sum())
        if slots >= n:
            assert stats["steps"] == int(w.dec_lens.max())
        # the handle goes back to batch operation
        sub = w.subset([0, 3])
        dec2_enc = dec.upload_encoder(sub.enc)
        if slots >= 2:
            dec.precompute_cross_kv(dec2_enc, sub.enc_lens)
            toks, lens = dec.greedy_decode(sub.dec_lens)
            toks = toks.cpu().numpy()
            for i, u in enumerate([0, 3]):
                for t in range(int(w.dec_lens[u])):
                    if ref["margin"][u, t] <= MARGIN:
                        break
                    assert toks[i, t] == ref["next"][u, t]
    finally:
        dec.close()


def test_stream_with_end_of_sequence():
    """With an end-of-sequence id the host learns from the slot lengths which slots are free."""
    from paper_2503_05931_b200 import binding, streaming
    n, slots = 17, 4
    w0, ref0 = _stream("bf16", n, seed=77)
    # an id whose first (clearly decided) occurrence lies in the middle of several utterances' free-running decodes
    first = {}
    for u in range(n):
        for t in range(int(w0.dec_lens[u])):
            if ref0["margin"][u, t] <= MARGIN:
                break
            first.setdefault(int(ref0["next"][u, t]), {}).setdefault(u, t)
    eos = max(first, key=lambda k: sum(t for u, t in first[k].items() if 2 <= t < int(w0.dec_lens[u]) - 1))
    w, ref = _stream("bf16", n, seed=77, eos=eos)
    assert (ref["lens"] < w.dec_lens).any()
    dec = binding.Decoder(w.model, w.weights, "bf16", max_batch=slots, max_total_enc_frames=slots * 150, max_enc_len=150,
                          max_dec_len=40, eos_id=eos)
    try:
        out, stats = streaming.decode_stream(dec, dec.upload_encoder(w.enc), w.enc_lens, w.dec_lens, slots, poll_steps=3)
        compared = 0
        for u in range(n):
            decided = True
            for t in range(int(ref["lens"][u])):
                if ref["margin"][u, t] <= MARGIN:
                    decided = False
                    break
                assert out[u][t] == ref["next"][u, t], (u, t)
                compared += 1
            if decided:
                assert len(out[u]) == int(ref["lens"][u]), (u, len(out[u]), int(ref["lens"][u]))
        print(f"[parity] stream with eos={eos}: {compared} greedy tokens compared, {stats}")
        assert compared > 3 * n
        assert stats["steps"] < int(w.dec_lens.sum())
    finally:
        dec.close()


def test_slot_argument_errors():
    import torch
    from paper_2503_05931_b200 import binding
    w = wl.make_custom(MID, [20, 30], [4, 4], dtype="bf16", seed=3)
    dec = binding.Decoder(w.model, w.weights, "bf16", max_batch=4, max_total_enc_frames=100, max_enc_len=30, max_dec_len=8)
    try:
        enc = dec.upload_encoder(w.enc)
        toks = torch.zeros((4, 8), dtype=torch.int32, device="cuda:0")
        lens = torch.zeros(4, dtype=torch.int32, device="cuda:0")
        for call, status in [(lambda: dec.admit(0, enc[:20], 4), binding.AED_ERR_STATE),          # no slots opened
                             (lambda: dec.greedy_steps(1, toks, lens), binding.AED_ERR_STATE),
                             (lambda: dec.open_slots(5), binding.AED_ERR_CAPACITY),              # > max_batch
                             (lambda: dec.open_slots(4), binding.AED_ERR_CAPACITY),              # 4 x 30 frames > 100
                             (lambda: dec.open_slots(0), binding.AED_ERR_INVALID_ARG)]:
            with pytest.raises(binding.AedError) as e:
                call()
            assert e.value.status == status
        dec.open_slots(3)
        assert dec.greedy_steps(5, toks, lens) == 0                 # nothing admitted: no step issued
        for call, status in [(lambda: dec.admit(3, enc[:20], 4), binding.AED_ERR_INVALID_ARG),
                             (lambda: dec.admit(0, enc[:50], 4), binding.AED_ERR_CAPACITY),
                             (lambda: dec.admit(0, enc[:20], 9), binding.AED_ERR_CAPACITY),
                             (lambda: dec.admit(0, enc[:20], 0), binding.AED_ERR_INVALID_ARG),
                             (lambda: dec.step(lens), binding.AED_ERR_STATE)]:
            with pytest.raises(binding.AedError) as e:
                call()
            assert e.value.status == status
        dec.admit(0, enc[:20], 4, lens)
        with pytest.raises(binding.AedError) as e:
            dec.admit(0, enc[20:50], 4, lens)                       # still decoding
        assert e.value.status == binding.AED_ERR_STATE
        assert dec.greedy_steps(10, toks, lens) == 4
        dec.sync_status()
        assert lens.cpu().tolist() == [4, 0, 0, 0]
        dec.admit(0, enc[20:50], 2, lens)                           # free again
        assert dec.greedy_steps(10, toks, lens) == 2
        dec.sync_status()
        assert lens.cpu().tolist() == [2, 0, 0, 0]
    finally:
        dec.close()
