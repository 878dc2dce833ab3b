"""Prompt prefill (several positions per utterance in one batched causal pass) against the CPU checker run on the same
forced prefix: logits of the last prompt position, the greedy choice, and the steps that follow (they read the
keys and values the prefill cached)."""
import numpy as np
import pytest

from oracle import aed_oracle as orc
from paper_2503_05931_b200 import workloads as wl
from tests.helpers import MARGIN, TOL

pytestmark = pytest.mark.gpu

MID = dict(n_layers=3, d_model=256, n_heads=4, d_ffn=512, vocab=1000, d_enc=192)


@pytest.mark.parametrize("prompt_len,max_batch", [(5, 64), (5, 13), (5, 6), (1, 6), (19, 200)])
def test_prefill_matches_the_checker(prompt_len, max_batch):
    """max_batch 64 / 200: the whole prompt in one pass; 13: chunks of two positions (2 + 2 + 1); 6 = batch: one
    position per pass, i.e. plain steps."""
    import torch
    from paper_2503_05931_b200 import binding
    enc_lens = [40, 7, 130, 1, 66, 23]
    B, follow = len(enc_lens), 4
    L = prompt_len + follow
    w = wl.make_custom(MID, enc_lens, [L] * B, dtype="bf16", seed=55, out_std=0.1, ln_std=0.2)
    rng = np.random.default_rng(prompt_len * 100 + max_batch)
    forced = rng.integers(0, MID["vocab"], size=(B, L)).astype(np.int32)
    ref = orc.decode_batch(orc.Model(w.model, w.weights), w.enc, w.enc_lens, [L] * B, forced=forced, want_logits=True)
    dec = binding.Decoder(w.model, w.weights, "bf16", max_batch=max_batch, max_total_enc_frames=int(sum(enc_lens)),
                          max_enc_len=max(enc_lens), max_dec_len=L)
    try:
        dec.precompute_cross_kv(dec.upload_encoder(w.enc), w.enc_lens)
        logits = torch.full((B, MID["vocab"]), float("nan"), dtype=torch.float32, device="cuda:0")
        nxt = torch.full((B,), -1, dtype=torch.int32, device="cuda:0")
        prompt = torch.from_numpy(np.ascontiguousarray(forced[:, :prompt_len])).to("cuda:0")
        dec.prefill(prompt, logits, nxt)
        worst, compared = 0.0, 0
        for t in range(prompt_len - 1, L):
            if t >= prompt_len:
                dec.step(torch.from_numpy(np.ascontiguousarray(forced[:, t])).to("cuda:0"), None, logits, nxt)
            got, got_next = logits.cpu().numpy(), nxt.cpu().numpy()
            for u in range(B):
                worst = max(worst, float(np.max(np.abs(got[u] - ref["logits"][u][t]))))
                if ref["margin"][u, t] > MARGIN:
                    assert got_next[u] == ref["next"][u, t], (u, t)
                    compared += 1
        dec.sync_status()
        print(f"[parity] prefill P={prompt_len} max_batch={max_batch}: max |logit diff| = {worst:.3e}, {compared} argmax compared")
        assert worst < TOL["bf16"]
        assert compared > 0
        with pytest.raises(binding.AedError) as e:
            dec.prefill(prompt)                     # not directly after a precompute
        assert e.value.status == binding.AED_ERR_STATE
    finally:
        dec.close()


def test_prefill_argument_errors():
    import torch
    from paper_2503_05931_b200 import binding
    w = wl.make_custom(MID, [5, 9], [4, 4], dtype="bf16", seed=1)
    dec = binding.decoder_for_workload(w)
    prompt = torch.ones((2, 5), dtype=torch.int32, device="cuda:0")
    with pytest.raises(binding.AedError) as e:
        dec.prefill(prompt)
    assert e.value.status == binding.AED_ERR_STATE              # no batch yet
    dec.precompute_cross_kv(dec.upload_encoder(w.enc), w.enc_lens)
    with pytest.raises(binding.AedError) as e:
        dec.prefill(prompt)
    assert e.value.status == binding.AED_ERR_CAPACITY           # 5 positions, max_dec_len 4
    dec.close()
    w32 = wl.make_custom(MID, [5, 9], [4, 4], dtype="fp32", seed=1)
    dec = binding.decoder_for_workload(w32)
    dec.precompute_cross_kv(dec.upload_encoder(w32.enc), w32.enc_lens)
    with pytest.raises(binding.AedError) as e:
        dec.prefill(prompt[:, :2].contiguous())
    assert e.value.status == binding.AED_ERR_UNSUPPORTED
    dec.close()
