"""The paper's 2D bucketing on the synthetic length law: 30 duration bins of equal cumulative-duration occupancy x 2
token sub-bins, estimated on a separate sample, strict and flexible allocation (Sections "Methods" and
"Experimental setup").  The paper reports 57 % / 59 % padding for fixed batches padded to 40 s against 4.5 % / 19 %
with 30x2 buckets on its own data; the synthetic law must show the same direction and order of magnitude."""
import numpy as np

from paper_2503_05931_b200 import bucketing, workloads


def _lengths(seed, n):
    rng = np.random.default_rng(seed)
    _, enc, dec = workloads.draw_lengths(rng, n, "lognormal")
    return enc, dec


def test_bins_have_equal_cumulative_duration():
    enc, dec = _lengths(1, 20000)
    dur_bounds, tok_bounds = bucketing.estimate_bins_2d(enc, dec, 30, 2)
    assert dur_bounds.shape == (30,) and tok_bounds.shape == (30, 2)
    assert np.all(np.diff(dur_bounds) >= 0) and dur_bounds[-1] == enc.max()
    which = np.searchsorted(dur_bounds, enc, side="left")
    mass = np.bincount(which, weights=enc, minlength=30)
    # equal occupancy in frames; the durations clipped to 40 s pile up on the last bound, which the last bins share
    body = mass[:27]
    assert body.max() / body.mean() < 1.25 and body.min() / body.mean() > 0.75
    assert abs(mass[27:].sum() / (3 * body.mean()) - 1) < 0.25
    counts = np.bincount(which, minlength=30)
    assert counts[0] > 3 * counts[26]                                               # hence many more short utterances per bin
    assert np.all(tok_bounds[:, 0] <= tok_bounds[:, 1])


def test_strict_discards_what_flexible_keeps():
    est_enc, est_dec = _lengths(2, 5000)          # the estimation sample ...
    enc, dec = _lengths(3, 4096)                  # ... is not the data that is bucketed
    dur_bounds, tok_bounds = bucketing.estimate_bins_2d(est_enc, est_dec, 30, 2)
    strict = bucketing.allocate_to_buckets(enc, dec, dur_bounds, tok_bounds, "strict")
    flexible = bucketing.allocate_to_buckets(enc, dec, dur_bounds, tok_bounds, "flexible")
    assert np.sum(strict < 0) > 0                                        # transcripts above their bin's bound are dropped
    assert np.sum(flexible < 0) < np.sum(strict < 0)
    kept = strict >= 0
    assert np.array_equal(strict[kept], flexible[kept])                  # where strict finds a bucket, flexible finds the same
    moved = (strict < 0) & (flexible >= 0)
    assert np.all(flexible[moved] // 2 > np.searchsorted(dur_bounds, enc[moved], side="left"))   # into a bin of longer utterances
    for u in np.flatnonzero(flexible >= 0):                              # every kept sample fits its bucket
        b, k = divmod(int(flexible[u]), 2)
        assert enc[u] <= dur_bounds[b] and dec[u] <= tok_bounds[b, k]
    # a sample nothing can hold is discarded in both modes
    far = bucketing.allocate_to_buckets(np.array([dur_bounds[-1] + 1]), np.array([1]), dur_bounds, tok_bounds, "flexible")
    assert far[0] == -1


def test_padding_goes_the_way_the_paper_reports():
    est_enc, est_dec = _lengths(4, 20000)
    enc, dec = _lengths(5, 4096)
    fixed = bucketing.fixed_batches(len(enc), 128)
    pe_f, pd_f = bucketing.padding_fractions_to(enc, dec, fixed, enc_to=500, dec_to=240)      # every batch padded to 40 s
    assert pe_f > 0.5 and pd_f > 0.5
    dur_bounds, tok_bounds = bucketing.estimate_bins_2d(est_enc, est_dec, 30, 2)
    sizes = bucketing.bucket_batch_sizes(dur_bounds, tok_bounds)
    batches, dropped = bucketing.bucket_batches(enc, dec, dur_bounds, tok_bounds, sizes, "flexible")
    assert len(dropped) <= 4 and sum(len(b) for b in batches) + len(dropped) == len(enc)
    pe_b, pd_b = bucketing.padding_fractions(enc, dec, batches)
    assert pe_b < 0.08 and pd_b < 0.30 and pe_b < pd_b                   # audio padding all but gone, transcripts harder
    pe_1, pd_1 = bucketing.padding_fractions(enc, dec, bucketing.bucket_batches(
        enc, dec, *bucketing.estimate_bins_2d(est_enc, est_dec, 30, 1), bucketing.bucket_batch_sizes(
            *bucketing.estimate_bins_2d(est_enc, est_dec, 30, 1)), "flexible")[0])
    assert pd_b < pd_1                                                   # the token sub-bins are what cuts transcript padding
    for b, batch in zip(range(len(batches)), batches):
        assert len(batch) >= 1
