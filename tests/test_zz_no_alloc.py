"""`ones_select_top_noalloc` against `ones_select_top`.

The no-allocation entry point serves callers that cannot obtain device memory when they run (the
device is already owned by a framework's allocator, or an allocation's device-wide synchronisation
does not fit their latency budget); its scratch is a fixed array inside the library.  The check:
through the C ABI, on calls in a row that share that array, its indices equal those of the entry
point that takes caller-provided scratch (integer indices: equality, as in the other selection
tests).  This file sorts last so that a run that stops at the first failure has already run every
other test; it also passes on its own in a fresh process.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _scores(n, seed):
    rng = np.random.default_rng(seed)
    f = rng.integers(0, max(2, n // 4), size=n).astype(np.float64) * 0.5 - 3.0  # many ties
    return torch.from_numpy(f).cuda()


def test_noalloc_selection_matches_scratch_version_on_consecutive_calls():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2108_03645_b200 import binding
    big, small = _scores(200_000, 1), _scores(777, 2)
    out = torch.empty(binding.NOALLOC_MAX_TOP, dtype=torch.int32, device="cuda")
    # calls back to back on the same stream: each finds the previous one's records in the array
    for scores, e in ((big, 64), (small, 5), (big, 1), (small, 64)):
        want = binding.select_top(scores, e)
        out.fill_(-7)
        got = binding.select_top_noalloc(scores, e, out)[:e]
        assert torch.equal(got, want), (scores.numel(), e)
        assert int(out[e:].ne(-7).sum()) == 0  # nothing written past e
    torch.cuda.synchronize()


def test_noalloc_selection_rejects_sizes_beyond_its_scratch():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2108_03645_b200 import binding
    scores = _scores(1000, 3)
    out = torch.empty(128, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.OnesError) as err:
        binding.select_top_noalloc(scores, binding.NOALLOC_MAX_TOP + 1, out)
    assert err.value.code == -5
    with pytest.raises(binding.OnesError) as err:
        binding.select_top_noalloc(scores[:3], 4, out)
    assert err.value.code == -3


def test_noalloc_selection_on_a_stream_of_the_callers():
    """The entry point enqueues on the stream it is given; a caller's own stream (not the default one) must see
    the same result, again on two calls in a row."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2108_03645_b200 import binding
    scores = _scores(50_000, 4)
    want = binding.select_top(scores, 7)
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    out = torch.full((binding.NOALLOC_MAX_TOP,), -7, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        for _ in range(2):
            got = binding.select_top_noalloc(scores, 7, out)[:7]
            stream.synchronize()
            assert torch.equal(got, want)
