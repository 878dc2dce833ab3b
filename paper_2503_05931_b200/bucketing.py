"""Host-side batching of an utterance stream: random batches versus 2D buckets.

The paper's central observation is that padding on two axes (input frames and output
tokens) wastes more than half of the computation, and that stratifying batches on both
lengths removes most of it (Sections "2D bucketing" and "Results", padding percentages
of the fixed-batch and 30x2-bucket runs).  For the decoder this matters through row
occupancy: every decode step streams all weights once, so the fewer steps a batch
spends with most rows already finished, the fewer weight re-streams per token.
"""
from __future__ import annotations

from typing import List

import numpy as np

def random_batches(n_utts: int, batch: int, rng: np.random.Generator) -> List[np.ndarray]:
    perm = rng.permutation(n_utts)
    return [perm[i:i + batch] for i in range(0, n_utts, batch)]


def bucket_batches_2d(enc_lens: np.ndarray, dec_lens: np.ndarray, n_enc_bins: int = 8, n_dec_bins: int = 4,
                      budget: int = 65536, max_batch: int = 2048) -> List[np.ndarray]:
    """2D bucketing: equal-count bins on encoder length, then equal-count sub-bins on output length.

    Follows the paper's strict 2D scheme (Section "2D bucketing": bucket on the input length first,
    then sub-bucket on the output length) with quantile bin edges estimated on the very utterances
    being bucketed, so no utterance is discarded.  The batch size of a bucket is the largest one
    whose padded footprint batch x (max T + max L) stays within ``budget`` frame+token units.
    """
    n = len(enc_lens)
    order = np.lexsort((dec_lens, enc_lens))       # by encoder length, ties by output length
    batches: List[np.ndarray] = []
    for eb in np.array_split(order, n_enc_bins):
        if len(eb) == 0:
            continue
        eb = eb[np.argsort(dec_lens[eb], kind="stable")]
        for db in np.array_split(eb, n_dec_bins):
            if len(db) == 0:
                continue
            foot = int(enc_lens[db].max()) + int(dec_lens[db].max())
            bsz = max(1, min(max_batch, budget // foot))
            for i in range(0, len(db), bsz):
                batches.append(db[i:i + bsz])
    assert sum(len(b) for b in batches) == n
    return batches


def padding_fractions(enc_lens: np.ndarray, dec_lens: np.ndarray, batches: List[np.ndarray]):
    """Share of a padded [batch, max length] rectangle that is padding, on both length axes."""
    enc_real = sum(int(enc_lens[b].sum()) for b in batches)
    dec_real = sum(int(dec_lens[b].sum()) for b in batches)
    enc_pad = sum(len(b) * int(enc_lens[b].max()) for b in batches)
    dec_pad = sum(len(b) * int(dec_lens[b].max()) for b in batches)
    return 1.0 - enc_real / enc_pad, 1.0 - dec_real / dec_pad
