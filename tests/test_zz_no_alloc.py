"""kvc_prefill_chunk_static: the entry point for callers that cannot allocate device memory
(code inside a pool that owns the device, plugins restricted to the buffers they are handed,
loops where an allocation would stall the GPU).  Its scratch is an array built into the library
instead of a caller-provided workspace, so here it is checked, through the C ABI, against
kvc_prefill_chunk on the same inputs: two calls in a row (the second one evicts), identical
attention output and identical cache afterwards.  Collected last on purpose."""
import ctypes

import pytest
import torch

from paper_2604_16734_b200 import binding
from paper_2604_16734_b200.binding import Kvc, KvcError, KVC_EINVAL

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,hq,hkv,d", [(torch.bfloat16, 8, 2, 128), (torch.float32, 4, 1, 64)])
def test_static_scratch_matches_workspace_entry_point(dtype, hq, hkv, d):
    torch.manual_seed(123)
    budget, chunk = 192, 160
    ref = Kvc(1, hq, hkv, d, dtype, budget, chunk, 16)
    sta = Kvc(1, hq, hkv, d, dtype, budget, chunk, 16)
    # the array keeps whatever the previous user left (the other parametrisation, other tests): the entry
    # point must not depend on it
    p = 0
    for n in (160, 150):                      # second call: 160 + 150 > 192 -> score, select, compact
        q = torch.randn(n, hq, d, device="cuda").to(dtype)
        k = torch.randn(n, hkv, d, device="cuda").to(dtype)
        v = torch.randn(n, hkv, d, device="cuda").to(dtype)
        out_ref = ref.prefill_chunk(0, q, k, v, p)
        out_sta = sta.prefill_chunk_static(0, q, k, v, p)
        torch.cuda.synchronize()
        assert ref.status() == 0 and sta.status_static() == 0
        tol = 1e-4 if dtype == torch.float32 else 2e-2
        assert (out_ref.float() - out_sta.float()).abs().max().item() <= tol
        p += n
    # a warm call allocates nothing: the free device memory is the same before and after it (inputs made up front)
    n = 40
    q = torch.randn(n, hq, d, device="cuda").to(dtype)
    k = torch.randn(n, hkv, d, device="cuda").to(dtype)
    v = torch.randn(n, hkv, d, device="cuda").to(dtype)
    out = torch.empty_like(q)
    out_ref = ref.prefill_chunk(0, q, k, v, p)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    sta.prefill_chunk_static(0, q, k, v, p, out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    assert sta.status_static() == 0
    assert (out_ref.float() - out.float()).abs().max().item() <= tol
    Kr, Vr, Pr, lr = ref.cache_view(0)
    Ks, Vs, Ps, ls = sta.cache_view(0)
    assert lr == ls == budget
    assert torch.equal(Pr[:, :lr], Ps[:, :ls])
    assert torch.equal(Kr[:, :lr], Ks[:, :ls]) and torch.equal(Vr[:, :lr], Vs[:, :ls])


def test_static_scratch_rejects_oversized_configuration():
    big = Kvc(1, 64, 64, 128, torch.bfloat16, 8192, 4096, allocate=False)      # needs > 1 MiB of scratch
    big.cache = torch.zeros(1, 256, dtype=torch.uint8, device="cuda")          # never touched: the size check comes first
    x = torch.zeros(8, 64, 128, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(KvcError) as e:
        big.prefill_chunk_static(0, x, x, x, 0)
    assert e.value.code == KVC_EINVAL and "scratch" in str(e.value)


def test_static_scratch_rejected_call_enqueues_nothing():
    # a call that fails its argument checks launches nothing (the clear of the shared status word included:
    # it is enqueued only after the checks) and leaves the context usable
    kvc = Kvc(1, 4, 2, 128, torch.bfloat16, 64, 32)
    x = torch.zeros(8, 4, 128, device="cuda", dtype=torch.bfloat16); y = torch.zeros(8, 2, 128, device="cuda", dtype=torch.bfloat16)
    kvc.prefill_chunk_static(0, x, y, y, 0)
    assert kvc.status_static() == 0
    before = kvc.launch_count()
    big = torch.zeros(40, 4, 128, device="cuda", dtype=torch.bfloat16); bigk = torch.zeros(40, 2, 128, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(KvcError) as e:
        kvc.prefill_chunk_static(0, big, bigk, bigk, 8)            # n > max_chunk
    assert e.value.code == KVC_EINVAL
    assert kvc.launch_count() == before and kvc.status_static() == 0
