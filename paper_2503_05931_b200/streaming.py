"""Continuous batching over a stream of utterances.

A static batch thins out until its longest utterance ends; with slots that are refilled in the step after their
utterance left, steps keep (nearly) all rows occupied without sorting the stream by output lengths that are not known
before decoding (the paper counts padded positions as wasted computation: Introduction, "Methods").  The scheduler
itself is ``aed_dec_decode_stream`` in the library; this module only shapes its arguments and results.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np


def decode_stream(dec, enc_packed, enc_lens: Sequence[int], max_lens: Sequence[int], slots: int, *,
                  poll_steps: int = 8, order: Optional[Sequence[int]] = None,
                  tokens_out=None, out_lens=None) -> Tuple[List[np.ndarray], dict]:
    """Greedy-decode every utterance of a stream through ``slots`` decoder slots.

    ``enc_packed``: device tensor [sum(enc_lens), d_enc] (utterance u at rows off[u] .. off[u+1]) in the handle's
    dtype; ``max_lens``: forced output lengths (upper bounds when the handle has an end-of-sequence id, in which case
    the slot lengths are read back every ``poll_steps`` steps); ``order``: arrival order (default 0, 1, 2, ...).

    Returns (tokens per utterance as int32 arrays, {"steps", "row_steps", "occupancy"}).
    """
    toks, lens, steps, row_steps = dec.decode_stream(enc_packed, enc_lens, max_lens, slots, order=order,
                                                     poll_steps=poll_steps, tokens_out=tokens_out, out_lens=out_lens)
    lens_np = lens.numpy()
    out = [toks[u, :int(lens_np[u])].numpy().copy() for u in range(len(lens_np))]
    return out, {"steps": steps, "row_steps": row_steps, "occupancy": row_steps / max(steps * slots, 1)}
