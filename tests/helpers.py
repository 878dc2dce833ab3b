"""Shared helpers of the GPU parity tests: drive the C ABI and compare with the CPU checker."""
import numpy as np

from oracle import aed_oracle as orc

TOL = {"fp32": 1e-4, "bf16": 3e-2}       # max-abs tolerance on teacher-forced logits
MARGIN = 0.1                             # greedy ids must match where the checker's top-2 margin exceeds this


def oracle_reference(w, rows=None, want_logits=True, n_threads=0, eos=-1, cross_kv_e4m3=False):
    """Free-running greedy decode of the given utterances (default: all) by the CPU checker."""
    sub = w if rows is None else w.subset(rows)
    model = orc.Model(w.model, w.weights, ln_eps=w.ln_eps, cross_kv_e4m3=cross_kv_e4m3)
    return orc.decode_batch(model, sub.enc, sub.enc_lens, sub.dec_lens, bos=w.bos_id, want_logits=want_logits,
                            n_threads=n_threads, eos=eos)


def comparable_tokens(w, ref, rows=None):
    """How many greedy tokens the checker fixes: per utterance, the steps before its first near-tie."""
    rows = list(range(w.batch)) if rows is None else [int(r) for r in rows]
    n = 0
    for i, u in enumerate(rows):
        for t in range(int(w.dec_lens[u])):
            if ref["margin"][i, t] <= MARGIN:
                break
            n += 1
    return n


def teacher_forced_compare(dec, w, ref, rows=None, check_rows_only=True):
    """Feed the checker's greedy tokens to aed_dec_step and compare logits and argmax at every step.

    ``ref`` covers the utterances ``rows`` (default all); the other utterances of the batch run on their own
    previous argmax.  Returns (max |logit diff|, number of compared argmax, mismatches with margin > MARGIN)."""
    import torch
    B, V = w.batch, w.model["vocab"]
    rows = list(range(B)) if rows is None else [int(r) for r in rows]
    Lmax = int(w.dec_lens.max())
    enc = dec.upload_encoder(w.enc)
    dec.precompute_cross_kv(enc, w.enc_lens)
    logits = torch.full((B, V), float("nan"), dtype=torch.float32, device=dec.device)
    nxt = torch.full((B,), w.bos_id, dtype=torch.int32, device=dec.device)
    toks = torch.full((B,), w.bos_id, dtype=torch.int32, device=dec.device)
    worst, compared, bad = 0.0, 0, []
    ridx = torch.tensor(rows, dtype=torch.long, device=dec.device)
    for t in range(Lmax):
        act = torch.from_numpy((w.dec_lens > t).astype(np.uint8)).to(dec.device)
        if t > 0:
            toks.copy_(nxt)
            forced = np.array([max(int(ref["next"][i, min(t, int(w.dec_lens[u])) - 1]), 0) for i, u in enumerate(rows)],
                              np.int32)
            toks[ridx] = torch.from_numpy(forced).to(dec.device)
        dec.step(toks, act, logits, nxt)
        got = logits[ridx].cpu().numpy()
        got_next = nxt[ridx].cpu().numpy()
        for i, u in enumerate(rows):
            if t >= int(w.dec_lens[u]):
                continue
            diff = float(np.max(np.abs(got[i].astype(np.float64) - ref["logits"][i][t])))
            worst = max(worst, diff)
            compared += 1
            if ref["margin"][i, t] > MARGIN and got_next[i] != ref["next"][i, t]:
                bad.append((u, t, int(got_next[i]), int(ref["next"][i, t])))
    dec.sync_status()
    return worst, compared, bad


def greedy_compare(dec, w, ref, rows=None):
    """aed_dec_greedy_decode against the checker: per utterance, tokens must agree up to and including the
    last step before the checker's first near-tie (margin <= MARGIN).  Returns the number of compared tokens."""
    rows = list(range(w.batch)) if rows is None else [int(r) for r in rows]
    enc = dec.upload_encoder(w.enc)
    dec.precompute_cross_kv(enc, w.enc_lens)
    toks, lens = dec.greedy_decode(w.dec_lens)
    toks, lens = toks.cpu().numpy(), lens.cpu().numpy()
    assert np.array_equal(lens, w.dec_lens)
    compared = 0
    for u in range(w.batch):
        L = int(w.dec_lens[u])
        assert np.all(toks[u, :L] >= 0) and np.all(toks[u, :L] < w.model["vocab"])
        assert np.all(toks[u, L:] == -1)
    for i, u in enumerate(rows):
        for t in range(int(w.dec_lens[u])):
            if ref["margin"][i, t] <= MARGIN:
                break
            assert toks[u, t] == ref["next"][i, t], f"utterance {u} step {t}: {toks[u, t]} vs {ref['next'][i, t]}"
            compared += 1
    assert compared == comparable_tokens(w, ref, rows)
    return compared, toks


def sinusoid(t, d):
    """PE(t) of the decoder's definition, written out with math.sin / math.cos."""
    import math
    pe = np.zeros(d)
    for i in range(0, d, 2):
        ang = t / (10000.0 ** (i / d))
        pe[i], pe[i + 1] = math.sin(ang), math.cos(ang)
    return pe


def torch_layer_logits(model, weights, enc, forced, ln_eps=1e-5):
    """Teacher-forced logits of one utterance from torch.nn.TransformerDecoderLayer(norm_first=True) in fp64, a final
    LayerNorm and a Linear: the library routine that pins the checker's layer."""
    import math
    import torch
    d, NL, L = model["d_model"], model["n_layers"], len(forced)
    t64 = lambda a: torch.tensor(np.asarray(a), dtype=torch.float64)
    x = torch.stack([t64(weights["embed"][y]) * math.sqrt(d) + t64(sinusoid(t, d)) for t, y in enumerate(forced)])[None]
    mem = t64(enc)[None]
    mask = torch.nn.Transformer.generate_square_subsequent_mask(L, dtype=torch.float64)
    with torch.no_grad():
        for l in range(NL):
            lay = torch.nn.TransformerDecoderLayer(d, model["n_heads"], model["d_ffn"], dropout=0.0, activation="relu",
                                                   batch_first=True, norm_first=True, dtype=torch.float64)
            lay.self_attn.in_proj_weight.copy_(t64(weights["w_qkv"][l])); lay.self_attn.in_proj_bias.copy_(t64(weights["b_qkv"][l]))
            lay.self_attn.out_proj.weight.copy_(t64(weights["w_o"][l])); lay.self_attn.out_proj.bias.copy_(t64(weights["b_o"][l]))
            lay.multihead_attn.in_proj_weight.copy_(t64(np.concatenate([weights["w_q_c"][l], weights["w_kv_c"][l]])))
            lay.multihead_attn.in_proj_bias.copy_(t64(np.concatenate([weights["b_q_c"][l], weights["b_kv_c"][l]])))
            lay.multihead_attn.out_proj.weight.copy_(t64(weights["w_o_c"][l])); lay.multihead_attn.out_proj.bias.copy_(t64(weights["b_o_c"][l]))
            lay.linear1.weight.copy_(t64(weights["w_ff1"][l])); lay.linear1.bias.copy_(t64(weights["b_ff1"][l]))
            lay.linear2.weight.copy_(t64(weights["w_ff2"][l])); lay.linear2.bias.copy_(t64(weights["b_ff2"][l]))
            for i, nm in ((1, "ln1"), (2, "ln2"), (3, "ln3")):
                getattr(lay, f"norm{i}").weight.copy_(t64(weights[nm + "_g"][l]))
                getattr(lay, f"norm{i}").bias.copy_(t64(weights[nm + "_b"][l]))
            x = lay.eval()(x, mem, tgt_mask=mask)
        x = torch.nn.functional.layer_norm(x, (d,), t64(weights["final_ln_g"]), t64(weights["final_ln_b"]), ln_eps)
        z = x @ t64(weights["w_out"]).T
        if weights.get("b_out") is not None:
            z = z + t64(weights["b_out"])
    return z[0].numpy()
