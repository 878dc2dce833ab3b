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


# ------------------------------------------------------------------------------------------------------------
# The paper's 2D bucketing as a host library (Sections "Methods: 2D bucketing" and "Experimental setup"):
# duration bins of equal occupancy in cumulative duration, estimated on a separate sample, each split into token
# sub-bins; strict and flexible sample-to-bucket allocation; one batch size per bucket.
# ------------------------------------------------------------------------------------------------------------
def _equal_mass_upper_bounds(values: np.ndarray, n_bins: int) -> np.ndarray:
    """Upper bounds of n_bins bins over ``values`` such that every bin holds the same share of sum(values)
    (the paper's "equal occupancy w.r.t. cumulative bin duration").  The last bound is the sample maximum."""
    v = np.sort(np.asarray(values, dtype=np.float64))
    if len(v) == 0:
        return np.zeros(0)
    cum = np.cumsum(v)
    targets = cum[-1] * np.arange(1, n_bins) / n_bins
    idx = np.searchsorted(cum, targets, side="left")
    bounds = np.concatenate([v[np.minimum(idx, len(v) - 1)], [v[-1]]])
    return np.maximum.accumulate(bounds)


def estimate_bins_2d(enc_lens: np.ndarray, dec_lens: np.ndarray, n_duration_bins: int = 30, n_token_bins: int = 2):
    """Bin estimation on a sample (the paper uses a 100k-utterance sample of the training data): ``n_duration_bins``
    upper bounds on the input length with equal cumulative-length occupancy, and inside every duration bin
    ``n_token_bins`` upper bounds on the output length, estimated the same way on the sample's members of that bin
    (the paper does not say how the token sub-bins are cut; equal cumulative-token occupancy mirrors its duration
    rule).  Returns (duration_bounds [D], token_bounds [D, K]); a bin without sample members inherits the bounds of
    the previous one."""
    enc_lens = np.asarray(enc_lens)
    dec_lens = np.asarray(dec_lens)
    dur_bounds = _equal_mass_upper_bounds(enc_lens, n_duration_bins)
    tok_bounds = np.zeros((len(dur_bounds), n_token_bins))
    lower = -np.inf
    for i, ub in enumerate(dur_bounds):
        members = dec_lens[(enc_lens > lower) & (enc_lens <= ub)]
        if len(members):
            tok_bounds[i] = _equal_mass_upper_bounds(members, n_token_bins)
        elif i > 0:
            tok_bounds[i] = tok_bounds[i - 1]
        lower = ub
    return dur_bounds, tok_bounds


def allocate_to_buckets(enc_lens: np.ndarray, dec_lens: np.ndarray, dur_bounds: np.ndarray, tok_bounds: np.ndarray,
                        mode: str = "flexible") -> np.ndarray:
    """Bucket index (duration bin * K + token sub-bin) of every utterance, or -1 if it is discarded.

    strict   : the duration bin is the first whose bound covers the input length; inside it the first token
               sub-bin whose bound covers the output length; a transcript longer than the bin's last bound is
               discarded (the baseline algorithm the paper describes).
    flexible : the smallest bucket, in (duration, token) order, that fits both lengths, which may lie in a bin of
               longer utterances: some input padding is traded for keeping the outlier (the paper's modification)."""
    D, K = tok_bounds.shape
    out = np.full(len(enc_lens), -1, dtype=np.int64)
    first_bin = np.searchsorted(dur_bounds, enc_lens, side="left")
    for u, (T, L, b0) in enumerate(zip(enc_lens, dec_lens, first_bin)):
        if b0 >= D:
            continue                              # longer than anything seen during estimation
        last = b0 + 1 if mode == "strict" else D
        for b in range(b0, last):
            k = int(np.searchsorted(tok_bounds[b], L, side="left"))
            if k < K:
                out[u] = b * K + k
                break
    return out


def bucket_batch_sizes(dur_bounds: np.ndarray, tok_bounds: np.ndarray, budget: int = 65536, max_batch: int = 2048) -> np.ndarray:
    """One batch size per bucket: the largest whose padded footprint batch x (bound on T + bound on L) stays within
    ``budget`` frame+token units.  (The paper calibrates them with a memory-driven search, or with a 360 s cumulative
    duration threshold; a decoder that holds no activations for a backward pass is bounded by its K/V footprint.)"""
    D, K = tok_bounds.shape
    foot = dur_bounds[:, None] + tok_bounds
    return np.clip((budget // np.maximum(foot, 1)).astype(np.int64), 1, max_batch).reshape(D * K)


def bucket_batches(enc_lens: np.ndarray, dec_lens: np.ndarray, dur_bounds: np.ndarray, tok_bounds: np.ndarray,
                   batch_sizes: np.ndarray, mode: str = "flexible"):
    """Batches of utterance indices, bucket by bucket, and the indices that were discarded."""
    alloc = allocate_to_buckets(enc_lens, dec_lens, dur_bounds, tok_bounds, mode)
    batches: List[np.ndarray] = []
    for b in range(len(batch_sizes)):
        members = np.flatnonzero(alloc == b)
        for i in range(0, len(members), int(batch_sizes[b])):
            batches.append(members[i:i + int(batch_sizes[b])])
    return batches, np.flatnonzero(alloc < 0)


def fixed_batches(n_utts: int, batch: int) -> List[np.ndarray]:
    """Consecutive fixed-size batches (the paper's fixed-batch comparison run pads every one to the longest allowed
    utterance; see ``padding_fractions`` with ``pad_to``)."""
    idx = np.arange(n_utts)
    return [idx[i:i + batch] for i in range(0, n_utts, batch)]


def padding_fractions_to(enc_lens: np.ndarray, dec_lens: np.ndarray, batches: List[np.ndarray], enc_to: int, dec_to: int):
    """Padding shares when every batch is padded to fixed lengths (enc_to frames, dec_to tokens)."""
    n = sum(len(b) for b in batches)
    enc_real = sum(int(enc_lens[b].sum()) for b in batches)
    dec_real = sum(int(dec_lens[b].sum()) for b in batches)
    return 1.0 - enc_real / (n * enc_to), 1.0 - dec_real / (n * dec_to)
