"""Match search + draft gather on the GPU against the oracle, bit-exact (Sec. 3.1-3.2;
App. B.3 step 1)."""
import numpy as np
import pytest
import torch

from oracle import copyspec_oracle as O
from paper_2502_08923_b200 import binding as cs, inputs
from helpers import i32

pytestmark = pytest.mark.gpu


def _check(hist, lens, gamma, k, policy):
    B, stride = hist.shape
    mp, dr, dl = cs.cs_find_match(i32(hist), i32(lens), gamma, k, policy)
    torch.cuda.synchronize()
    mp, dr, dl = mp.cpu().numpy(), dr.cpu().numpy(), dl.cpu().numpy()
    for b in range(B):
        n = int(lens[b])
        p0 = O.find_match(hist[b], n, gamma, policy)
        draft = O.gather_draft(hist[b], n, p0, gamma, k)
        assert mp[b] == p0, (b, n, gamma, policy)
        assert dl[b] == len(draft)
        assert dr[b, :len(draft)].tolist() == draft
        assert (dr[b, len(draft):] == -1).all()


@pytest.mark.parametrize("gamma", [3, 5])
@pytest.mark.parametrize("policy", [cs.LATEST, cs.FIRST])
def test_search_workload_full_size(gamma, policy):
    """64 histories of 32,768 Zipf tokens with planted spans and the three kinds of tail."""
    hist, kinds, _ = inputs.match_search_histories()
    lens = np.full(64, 32768, dtype=np.int32)
    _check(hist, lens, gamma, 10, policy)


@pytest.mark.parametrize("gamma", [1, 2, 3, 4, 5, 6, 8])
def test_ragged_lengths_small_alphabet(gamma):
    rng = np.random.default_rng(gamma)
    B, stride = 37, 5000
    hist = rng.integers(0, 3, size=(B, stride), dtype=np.int32)
    lens = rng.integers(0, stride + 1, size=B).astype(np.int32)
    lens[:8] = [0, 1, 2 * gamma - 1, 2 * gamma, 2 * gamma + 1, stride, stride - 1, 7]
    for policy in (cs.LATEST, cs.FIRST):
        for k in (0, 1, 10, 20):
            _check(hist, lens, gamma, k, policy)


@pytest.mark.parametrize("stride", [9, 33, 4097, 8191, 20001])
def test_unaligned_rows_and_cluster_boundaries(stride):
    rng = np.random.default_rng(stride)
    B = 5
    hist = rng.integers(0, 4, size=(B, stride), dtype=np.int32)
    lens = np.array([stride, stride - 1, stride // 2, max(0, stride - 3), min(stride, 6)], dtype=np.int32)
    for gamma in (3, 5):
        _check(hist, lens, gamma, 10, cs.LATEST)
        _check(hist, lens, gamma, 10, cs.FIRST)


def test_match_only_at_chunk_edges():
    """A single occurrence placed at every position around the CTA / vector boundaries."""
    stride, gamma = 16384, 3
    spots = [0, 1, 3, 4, 1023, 1024, 4095, 4096, 4097, 8191, 8192, 12287, 12288, 16384 - 2 * 3 - 2, 16384 - 2 * 3]
    hist = np.arange(len(spots) * stride, dtype=np.int32).reshape(len(spots), stride) % 1000003 + 10
    for b, p in enumerate(spots):
        hist[b, -3:] = [1, 2, 3]
        hist[b, p:p + 3] = [1, 2, 3]
    lens = np.full(len(spots), stride, dtype=np.int32)
    for policy in (cs.LATEST, cs.FIRST):
        _check(hist, lens, gamma, 10, policy)
        mp, _, _ = cs.cs_find_match(i32(hist), i32(lens), gamma, 10, policy)
        assert mp.cpu().tolist() == spots


def test_empty_batch_and_bad_arguments():
    h = torch.zeros(0, 16, dtype=torch.int32, device="cuda")
    n = torch.zeros(0, dtype=torch.int32, device="cuda")
    cs.cs_find_match(h, n, 3, 10)
    h = torch.zeros(2, 16, dtype=torch.int32, device="cuda")
    n = torch.full((2,), 16, dtype=torch.int32, device="cuda")
    with pytest.raises(cs.CsError):
        cs.cs_find_match(h, n, 0, 10)
    with pytest.raises(cs.CsError):
        cs.cs_find_match(h, n, 9, 10)


# ---------------------------------------------------------------- gamma-gram index (Sec. 3.1)
def _check_index(idx, hist, lens, gamma, k):
    hd, ld = i32(hist), i32(lens)
    idx.cs_gram_index_update(hd, ld)
    for policy in (cs.LATEST, cs.FIRST):
        mp, dr, dl = idx.cs_find_match_indexed(hd, ld, k, policy)
        torch.cuda.synchronize()
        mp, dr, dl = mp.cpu().numpy(), dr.cpu().numpy(), dl.cpu().numpy()
        for b in range(hist.shape[0]):
            n = int(lens[b])
            p0 = O.find_match(hist[b], n, gamma, policy)
            draft = O.gather_draft(hist[b], n, p0, gamma, k)
            assert mp[b] == p0, (b, n, gamma, policy)
            assert dl[b] == len(draft) and dr[b, :len(draft)].tolist() == draft
            assert (dr[b, len(draft):] == -1).all()


@pytest.mark.parametrize("gamma", [1, 3, 5])
def test_index_grows_token_by_token_small_alphabet(gamma):
    """Small alphabets make every gram repeat and overlap its own key; histories grow by ragged
    amounts between lookups, as in the loop.  Every lookup equals the oracle's scan."""
    rng = np.random.default_rng(gamma)
    B, stride = 6, 300
    hist = rng.integers(0, 3, size=(B, stride), dtype=np.int32)
    hist[4] = np.arange(stride) % 7                 # periodic: the latest occurrence always overlaps the key
    hist[5] = 2                                      # constant
    idx = cs.GramIndex(B, stride, gamma)
    lens = np.zeros(B, dtype=np.int32)
    while lens.min() < stride:
        lens = np.minimum(stride, lens + rng.integers(0, 12, size=B)).astype(np.int32)
        _check_index(idx, hist, lens, gamma, 10)
    assert idx.cs_gram_index_status() == 0


@pytest.mark.parametrize("gamma", [3, 5])
def test_index_on_the_search_workload(gamma):
    """64 histories of 32,768 Zipf tokens with planted spans: bulk build, then the same answers
    as the scan kernel and the oracle."""
    hist, kinds, _ = inputs.match_search_histories()
    lens = np.full(64, 32768, dtype=np.int32)
    idx = cs.GramIndex(64, 32768, gamma)
    _check_index(idx, hist, lens, gamma, 10)
    hd, ld = i32(hist), i32(lens)
    for policy in (cs.LATEST, cs.FIRST):
        a = cs.cs_find_match(hd, ld, gamma, 10, policy)
        b = idx.cs_find_match_indexed(hd, ld, 10, policy)
        for x, y in zip(a, b):
            assert torch.equal(x, y)
    assert idx.cs_gram_index_status() == 0


def test_index_overflow_is_reported():
    rng = np.random.default_rng(0)
    hist = rng.integers(0, 1 << 20, size=(1, 4096), dtype=np.int32)
    idx = cs.GramIndex(1, 16, 3)                     # sized for 16 tokens, fed 4,096
    idx.cs_gram_index_update(i32(hist), i32([4096]))
    assert idx.cs_gram_index_status() == cs.CS_ERR_CAPACITY
