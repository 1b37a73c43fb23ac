"""The allocation-free top-k entry point against the regular one.

Some users of the library may not allocate device memory at all (they run inside a stream capture, or in a serving
loop that must never wait on the allocator).  ``ls_topk_select_static`` serves them from a fixed scratch array inside
the library.  This test calls it through the C ABI, twice in a row, and requires the same selection, bit for bit, as
``ls_predict`` produces from the same scores.  It is collected last (file name) so that a run that stops at the first
failure has already executed every other test, and it does not depend on anything those tests leave behind.
"""
import numpy as np
import pytest
import torch

from oracle import leanstream_oracle as orc
from paper_2609_03079_b200 import binding as ls
from paper_2609_03079_b200 import workload as wl

pytestmark = pytest.mark.gpu


def test_static_topk_matches_ls_predict_twice_in_a_row():
    dev = torch.device("cuda", 0)
    spec = wl.SPECS["tiny"]
    la = wl.make_layer(spec, 0)
    layer = ls.ls_layer_create(la, 0)
    toks = wl.make_tokens(spec)
    F = layer.d_ff
    idx = torch.full((F,), -1, dtype=torch.int32, device=dev)
    mask = torch.zeros((F + 31) // 32, dtype=torch.int32, device=dev)
    count = torch.zeros(1, dtype=torch.int32, device=dev)
    # two calls in a row, different inputs and sizes: the second must not see anything of the first in the scratch
    for call, (tok, k) in enumerate([(toks[0], spec.k), (toks[1], F)]):
        ref = ls.Selection(F, k, 0)
        ls.ls_predict(layer, torch.from_numpy(tok).to(dev), k, ref)
        idx.fill_(-1)
        ls.ls_topk_select_static(ref.scores, k, idx, mask, count)
        torch.cuda.synchronize()
        assert int(count.item()) == k == int(ref.count.item())
        assert torch.equal(idx[:k], ref.idx[:k]), f"call {call}: selected order differs"
        assert torch.equal(mask, ref.mask), f"call {call}: mask differs"
    # ties and special values follow the same total order as the regular entry point
    s = torch.tensor([1.0, 2.0, 2.0, -0.0, 0.0, float("nan"), 2.0], dtype=torch.float64, device=dev)
    ls.ls_topk_select_static(s, 7, idx, None, count)
    assert idx[:7].tolist() == [1, 2, 6, 0, 3, 4, 5]
    layer.close()


def test_static_topk_rejects_sizes_beyond_its_scratch():
    dev = torch.device("cuda", 0)
    big = torch.zeros(ls.LS_STATIC_TOPK_MAX_N + 1, dtype=torch.float64, device=dev)
    idx = torch.zeros(8, dtype=torch.int32, device=dev)
    count = torch.zeros(1, dtype=torch.int32, device=dev)
    with pytest.raises(ls.LeanStreamError) as e:
        ls.ls_topk_select_static(big, 4, idx, None, count)
    assert e.value.code == ls.LS_ERR_INVALID and str(ls.LS_STATIC_TOPK_MAX_N) in str(e.value)
    with pytest.raises(ls.LeanStreamError):
        ls.ls_topk_select_static(big[:16], 17, idx, None, count)


@pytest.mark.parametrize("n,k,kind", [(1024, 160, "normal"), (32768, 20000, "normal"), (32768, 5000, "coarse"), (4096, 1000, "equal")])
def test_static_topk_against_the_oracle(n, k, kind):
    """The allocation-free entry point against the oracle's total order itself, at its largest size (where the
    candidates no longer fit in shared memory and live in the static array), with heavy ties and with all scores equal."""
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(n + k)
    if kind == "normal":
        s = rng.standard_normal(n)
    elif kind == "coarse":
        s = np.round(rng.standard_normal(n) * 4.0) / 4.0  # about thirty distinct values: long runs of exact ties
    else:
        s = np.full(n, -1.5)
    idx = torch.full((n,), -1, dtype=torch.int32, device=dev)
    mask = torch.zeros((n + 31) // 32, dtype=torch.int32, device=dev)
    count = torch.zeros(1, dtype=torch.int32, device=dev)
    want = orc.topk_order(s, k)
    for _ in range(2):
        ls.ls_topk_select_static(torch.from_numpy(s).to(dev), k, idx, mask, count)
        torch.cuda.synchronize()
        assert int(count.item()) == k
        assert idx[:k].cpu().numpy().astype(np.int64).tolist() == want.tolist()
        assert np.array_equal(mask.cpu().numpy().view(np.uint32), orc.mask_of(want, n))
