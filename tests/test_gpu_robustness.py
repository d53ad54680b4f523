"""GPU tests of the corners around the hot path: the query-agnostic score on degenerate keys (Sec. 3.2: keys
parallel to the anchor, identical keys, a zero key), the bounded device-side wait running out, and the guard
regions that the parity helper keeps around every buffer."""
import numpy as np
import pytest
import torch

from oracle.kvc_oracle import KVCOracle
from paper_2604_16734_b200 import binding
from paper_2604_16734_b200.binding import Kvc, KVC_ETIMEOUT

from parity_util import check_guards, compare_chunk, guarded_copy, install_guards

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------------------------------------
# query-agnostic score (Sec. 3.2) where the cosine reaches 1: the keys the policy must evict first

def _parallel_keys(a, n, specials):
    """n keys per kv-head that are all positive power-of-two multiples of the direction a ([1][Hkv][d]; so every
    cosine to the anchor is exactly the same number in any precision), except the rows named in `specials`:
    'neg' = -a (the least similar key there can be), 'neg2' = -2a, 'zero' = the zero key."""
    scale = torch.tensor([1.0, 2.0, 0.5, 4.0])[torch.arange(n) % 4].view(n, 1, 1)
    k = (a.float() * scale).to(a.dtype)
    for row, kind in specials.items():
        k[row] = {"neg": -a[0], "neg2": (-2 * a[0].float()).to(a.dtype), "zero": torch.zeros_like(a[0])}[kind]
    return k.contiguous()


@pytest.mark.parametrize("dtype,d,hq,hkv", [(torch.float32, 64, 2, 1), (torch.float32, 128, 4, 2), (torch.bfloat16, 64, 4, 2),
                                            (torch.bfloat16, 128, 4, 1)])
@pytest.mark.parametrize("seed", [0, 1, 2, 3, 4, 5])
def test_query_agnostic_score_with_keys_parallel_to_the_anchor(dtype, d, hq, hkv, seed):
    # Every ordinary key is a positive multiple of a, so the anchor is parallel to a and 1 - cos rounds to zero or
    # to a few ulps on either side of it; the only dissimilar keys are -a (score 2), the zero key (score 1) and,
    # in the second block, -2a (score 2, younger than -a).  With two places for candidates the retained sets are
    # fixed: {-a, zero} after the first block, {-a, -2a} after the second.  The cut-off gap is about 1, so the
    # oracle's set has to be matched exactly.
    w, B, c = 4, 6, 40
    kvc = Kvc(1, hq, hkv, d, dtype, B, c, w, policy=binding.KVC_SCORE_KEYDIFF)
    orc = KVCOracle(1, hq, hkv, d, B, w, policy="keydiff")
    g = torch.Generator().manual_seed(100 + seed)
    a = torch.randn(1, hkv, d, generator=g).to(dtype)
    k1 = _parallel_keys(a, 40, {7: "neg", 21: "zero"})
    q1 = torch.randn(40, hq, d, generator=g).to(dtype); v1 = torch.randn(40, hkv, d, generator=g).to(dtype)
    compare_chunk(kvc, orc, 0, q1, k1, v1, 0)
    _, _, pos, ln = kvc.cache_view(0)
    for h in range(hkv):
        assert sorted(pos[h, :ln].tolist()) == [7, 21, 36, 37, 38, 39]
    k2 = _parallel_keys(a, 30, {11: "neg2"})
    q2 = torch.randn(30, hq, d, generator=g).to(dtype); v2 = torch.randn(30, hkv, d, generator=g).to(dtype)
    compare_chunk(kvc, orc, 0, q2, k2, v2, 40)
    _, _, pos, ln = kvc.cache_view(0)
    for h in range(hkv):
        assert sorted(pos[h, :ln].tolist()) == [7, 40 + 11, 66, 67, 68, 69]
    # no score may be negative: the selection orders scores by their bit patterns
    _, score = kvc.workspace_view(0)
    assert float(score[:, :32].min()) >= 0.0


@pytest.mark.parametrize("dtype,d", [(torch.float32, 64), (torch.bfloat16, 128)])
def test_query_agnostic_score_identical_keys_keep_the_oldest(dtype, d):
    # all keys identical: every candidate has exactly the same score, so the older entries stay (the tie rule),
    # whatever sign the rounding of 1 - cos takes
    hq = hkv = 2; w, B, c = 2, 9, 32
    for seed in range(6):
        kvc = Kvc(1, hq, hkv, d, dtype, B, c, w, policy=binding.KVC_SCORE_KEYDIFF)
        g = torch.Generator().manual_seed(300 + seed)
        a = torch.randn(1, hkv, d, generator=g).to(dtype)
        k = a.repeat(32, 1, 1).contiguous()
        q = torch.randn(32, hq, d, generator=g).to(dtype); v = torch.randn(32, hkv, d, generator=g).to(dtype)
        kvc.prefill_chunk(0, q.cuda(), k.cuda(), v.cuda(), 0)
        torch.cuda.synchronize()
        assert kvc.status() == 0
        _, _, pos, ln = kvc.cache_view(0)
        _, score = kvc.workspace_view(0)
        assert ln == B
        for h in range(hkv):
            assert sorted(pos[h, :ln].tolist()) == list(range(B - w)) + [30, 31]
            assert float(score[h, :30].min()) >= 0.0 and float(score[h, :30].max()) <= 1e-5


# ------------------------------------------------------------------------------------------------
# scores that leave the running maximum far behind

@pytest.mark.parametrize("hq,hkv,blocks", [(2, 2, (512, 512)), (8, 2, (256, 200, 256)), (4, 1, (128, 128, 128, 77))])
def test_a_key_whose_score_dwarfs_everything_before_it(hq, hkv, blocks):
    # The attention kernel keeps a reference maximum per row and raises it (rescaling O and the row sum) only when a
    # tile's maximum exceeds it by more than a threshold.  Here every query is the same +-1 vector u, ordinary keys
    # are small, and a few keys are large multiples of u, each larger than the last, placed in the first and in the
    # second half of key tiles that are not a row's first: their scores (5 |u|^2 / sqrt(d) = 57 nats and up) exceed
    # everything before them by far more than any lazy rule may let pass, for the rows that can see them and not for
    # the others of the same warp.  The softmax saturates on those keys; outputs, scores and retained sets must match.
    d, B, w = 128, 1024, 8
    kvc = Kvc(1, hq, hkv, d, torch.bfloat16, B, max(blocks), w)
    orc = KVCOracle(1, hq, hkv, d, B, w)
    g = torch.Generator().manual_seed(7)
    u = (torch.randint(0, 2, (d,), generator=g) * 2 - 1).float()
    big = {200: 5.0, 300: 8.0, 470: 12.0, 600: 16.0, 900: 24.0}     # token -> multiple of u (tile halves: 2nd, 1st, 2nd, 2nd, 1st)
    p = 0
    for n in blocks:
        q = u.expand(n, hq, d).clone().bfloat16()
        k = (0.25 * torch.randn(n, hkv, d, generator=g)).bfloat16()
        v = torch.randn(n, hkv, d, generator=g).bfloat16()
        for tok, mult in big.items():
            if p <= tok < p + n:
                k[tok - p] = (mult * u).bfloat16()
        stats = compare_chunk(kvc, orc, 0, q, k, v, p)
        assert kvc.status() == 0
        p += n
    assert stats is not None

# ------------------------------------------------------------------------------------------------
# the bounded wait

def test_a_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable():
    # Every wait in the kernels gives up after the context's limit.  The self-test kernel waits on a barrier that
    # nothing will ever complete, with a limit of about 64k cycles: it must return by itself, the status word must
    # read KVC_ETIMEOUT, and after the status word is cleared an ordinary block must run and match the oracle.
    hq, hkv, d = 4, 2, 128
    kvc = Kvc(1, hq, hkv, d, torch.bfloat16, 64, 48, 8)
    install_guards(kvc)
    kvc.set_wait_limit(1 << 16)
    kvc.selftest_wait_timeout()
    torch.cuda.synchronize()
    assert kvc.status() == KVC_ETIMEOUT
    assert "status word" in kvc.last_error()
    check_guards(kvc)
    kvc.workspace_init()
    assert kvc.status() == 0
    kvc.set_wait_limit(2_000_000_000)
    orc = KVCOracle(1, hq, hkv, d, 64, 8)
    torch.manual_seed(5)
    p = 0
    for n in (48, 40):
        q = torch.randn(n, hq, d).bfloat16(); k = torch.randn(n, hkv, d).bfloat16(); v = torch.randn(n, hkv, d).bfloat16()
        compare_chunk(kvc, orc, 0, q, k, v, p)
        p += n
    with pytest.raises(binding.KvcError):
        kvc.set_wait_limit(10)                       # below the accepted range


# ------------------------------------------------------------------------------------------------
# the guard regions themselves

def test_guard_check_notices_a_stray_byte():
    # the checker must fail when a byte outside a buffer changes (here: written by the test itself, on the host side
    # of the comparison, never by a kernel)
    kvc = Kvc(2, 2, 1, 64, torch.float32, 32, 16, 4)
    install_guards(kvc)
    check_guards(kvc)
    whole, view = guarded_copy(torch.zeros(5, 2, 64), kvc.device)
    check_guards(kvc, [(whole, view)])
    kvc._guards["cache"][kvc._guards["stride"] + 3] = 0          # inside the gap after blob 0
    with pytest.raises(AssertionError):
        check_guards(kvc)
    kvc._guards["cache"][kvc._guards["stride"] + 3] = 0xA5
    whole[-1] = 1
    with pytest.raises(AssertionError):
        check_guards(kvc, [(whole, view)])


# ------------------------------------------------------------------------------------------------
# device-side time stamps

@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_device_time_stamps_count_every_launch(dtype):
    # every kernel of the stamped calls leaves a record with begin <= end; the records' durations, added per kind,
    # fit inside the span from the first begin to the last end (the kernels run in stream order), and the results
    # are those of an unstamped run
    hq, hkv, d = 8, 2, 128
    a = Kvc(1, hq, hkv, d, dtype, 256, 160, 16)
    b = Kvc(1, hq, hkv, d, dtype, 256, 160, 16)
    torch.manual_seed(11)
    blocks = [(torch.randn(n, hq, d, device="cuda").to(dtype), torch.randn(n, hkv, d, device="cuda").to(dtype),
               torch.randn(n, hkv, d, device="cuda").to(dtype)) for n in (160, 150, 160, 33)]
    before = b.launch_count()
    b.profile_device(64)
    p = 0
    for q, k, v in blocks:
        oa = a.prefill_chunk(0, q, k, v, p); ob = b.prefill_chunk(0, q, k, v, p)
        assert torch.equal(oa, ob)
        p += q.shape[0]
    ms, cnt, span = b.profile_device_read()
    b.profile_device(0)
    assert sum(cnt.values()) == b.launch_count() - before
    assert cnt["attention"] == 4 and cnt["compress"] == 3
    assert all(ms[s] > 0 for s in cnt if cnt[s]) and sum(ms.values()) <= span * 1.001
    assert torch.equal(a.cache_view(0)[2], b.cache_view(0)[2])
    # off again: the next call must not touch the (freed) record buffer
    q, k, v = blocks[0]
    b.prefill_chunk(0, q, k, v, p)
    torch.cuda.synchronize()
    assert b.status() == 0
