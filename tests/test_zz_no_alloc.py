"""The allocation-free step variant.

Some callers of the library cannot allocate device memory (a memory pool frozen at start-up, a thread that may not
block in the driver, a runtime without an allocator), so aed_dec_step_static_scratch keeps the flash-decoding scratch in an array
built into the library.  It must give what aed_dec_step gives.  This file is collected last on purpose: a
run that stops at the first failure has then already run every other test."""
import numpy as np
import pytest

from paper_2503_05931_b200 import workloads as wl
from tests.helpers import TOL, oracle_reference

pytestmark = pytest.mark.gpu

MODEL = dict(n_layers=2, d_model=128, n_heads=2, d_ffn=256, vocab=300, d_enc=128)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_static_scratch_step_matches_step(dtype):
    """Only the fp32 configuration writes attention partials, so only there does the built-in array carry data
    (several 64-position chunks per row: 130 and 65 frames); the bf16 run checks that the call is a plain step."""
    import torch
    from paper_2503_05931_b200 import binding
    w = wl.make_custom(MODEL, [130, 7, 64, 65], [5, 5, 5, 5], dtype=dtype, seed=31)
    B, V = w.batch, MODEL["vocab"]
    dev = "cuda:0"

    def run(static: bool):
        dec = binding.decoder_for_workload(w)
        dec.precompute_cross_kv(dec.upload_encoder(w.enc), w.enc_lens)
        toks = torch.full((B,), w.bos_id, dtype=torch.int32, device=dev)
        nxt = torch.zeros(B, dtype=torch.int32, device=dev)
        out = []
        for t in range(3):          # consecutive calls share the array and must not disturb each other
            logits = torch.full((B, V), float("nan"), dtype=torch.float32, device=dev)
            (dec.step_static_scratch if static else dec.step)(toks, None, logits, nxt)
            toks = torch.full((B,), 5 + t, dtype=torch.int32, device=dev)
            out.append((logits.cpu().numpy(), nxt.cpu().numpy().copy()))
        dec.sync_status()
        dec.close()
        return out

    ref, got = run(False), run(True)
    for (rl, rn), (gl, gn) in zip(ref, got):
        assert np.all(np.isfinite(gl))
        assert np.max(np.abs(gl - rl)) <= TOL[dtype]
        assert np.array_equal(gn, rn)
    # and against the CPU checker, teacher-forced on the same inputs (bos, then 5, 6)
    from oracle import aed_oracle as orc
    model = orc.Model(w.model, w.weights, ln_eps=w.ln_eps)
    forced = np.array([[w.bos_id, 5, 6]] * B, np.int32)
    chk = orc.decode_batch(model, w.enc, w.enc_lens, [3] * B, forced=forced, want_logits=True)
    for t, (gl, _) in enumerate(got):
        for u in range(B):
            assert np.max(np.abs(gl[u] - chk["logits"][u][t])) <= TOL[dtype]


def test_static_scratch_chunk_stride_fp32():
    """fp32 rows with many chunks (a 300-frame encoder output, a decode past 64 positions): the partials of every
    (row, head, chunk) sit at their stride inside the shared array, two calls in a row, against the checker."""
    import torch
    from paper_2503_05931_b200 import binding
    w = wl.make_custom(MODEL, [300, 129, 1], [70, 70, 70], dtype="fp32", seed=32)
    ref = oracle_reference(w)
    B, V = w.batch, MODEL["vocab"]
    dec = binding.decoder_for_workload(w)
    dec.precompute_cross_kv(dec.upload_encoder(w.enc), w.enc_lens)
    toks = torch.full((B,), w.bos_id, dtype=torch.int32, device="cuda:0")
    logits = torch.zeros((B, V), dtype=torch.float32, device="cuda:0")
    worst = 0.0
    for t in range(70):
        dec.step_static_scratch(toks, None, logits, None)
        got = logits.cpu().numpy()
        worst = max(worst, max(float(np.max(np.abs(got[u] - ref["logits"][u][t]))) for u in range(B)))
        toks = torch.from_numpy(ref["next"][:, t].astype(np.int32)).to("cuda:0")
    dec.sync_status()
    dec.close()
    assert worst <= TOL["fp32"], worst


def test_static_scratch_rejects_oversized_batches():
    import torch
    from paper_2503_05931_b200 import binding
    lib = binding.load_library()
    limit = int(lib.aed_dec_static_scratch_bytes())
    assert limit == 8 << 20
    # 1100 utterances x 2 heads x ceil(960 / 64) chunks x 264 bytes is more than the built-in array holds
    assert 1100 * 2 * 15 * 264 > limit
    for dtype in ("fp32", "bf16"):
        w = wl.make_custom(MODEL, [960] + [1] * 1099, [1] * 1100, dtype=dtype, seed=1)
        dec = binding.decoder_for_workload(w)
        dec.precompute_cross_kv(dec.upload_encoder(w.enc), w.enc_lens)
        toks = torch.ones(1100, dtype=torch.int32, device="cuda:0")
        if dtype == "fp32":             # the configuration that writes partials: refused, nothing launched
            with pytest.raises(binding.AedError) as e:
                dec.step_static_scratch(toks)
            assert e.value.status == binding.AED_ERR_CAPACITY and "built-in array" in e.value.message
            dec.step(toks)              # the ordinary step still runs
        else:                           # bf16 writes no partials and is never refused on this ground
            dec.step_static_scratch(toks)
        dec.sync_status()
        dec.close()
