"""HBM neuron cache: logical state (resident sets, miss lists, execution order) bit-exact against the oracle's
LogicalCache, and values of cached steps against the oracle."""
import numpy as np
import pytest
import torch

from oracle import leanstream_oracle as orc
from paper_2609_03079_b200 import binding as ls
from paper_2609_03079_b200 import workload as wl
from tests.helpers import assert_values_close, mask_to_set

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=[ls.LS_MISS_PATH_GATHER, ls.LS_MISS_PATH_LANE], ids=["gather", "lane"])
def miss_path(request):
    """Every test runs on both transports of the misses: the gather kernel that reads pinned host memory itself, and the
    host I/O lane (a thread of the library polling the flags the decision kernels raise, copies by cudaMemcpyAsync)."""
    torch.cuda.synchronize()
    ls.ls_set_option(ls.LS_OPT_MISS_PATH, request.param)
    yield request.param
    torch.cuda.synchronize()
    ls.ls_set_option(ls.LS_OPT_MISS_PATH, ls.LS_MISS_PATH_GATHER)
DEV = 0


def dev_tensor(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda(DEV)


def snapshot(gl):
    m = torch.zeros(gl.nwords, dtype=torch.int32, device=f"cuda:{DEV}")
    ls.ls_cache_snapshot(gl, m)
    return mask_to_set(m.cpu().numpy().view(np.uint32), gl.d_ff)


def ar1_spec(seed=31, n_tokens=12, layers=1):
    return wl.StackSpec("cache-tiny", seed, layers, 256, 1024, True, "bf16", 32, 0.15, n_tokens, "ar1", ar_rho=0.8)


def test_reserve_trace_matches_oracle():
    spec = ar1_spec()
    la = wl.make_layer(spec, 0)
    C_ROWS, k = 300, 160
    gl = ls.ls_layer_create(la, DEV, cache_rows=C_ROWS)
    OL = orc.OracleLayer.from_arrays(la)
    cache = orc.LogicalCache(OL.d_ff, C_ROWS)
    sel = ls.Selection(gl.d_ff, k, DEV)
    slots = torch.empty(k, dtype=torch.int32, device=f"cuda:{DEV}")
    nhit = torch.zeros(1, dtype=torch.int32, device=f"cuda:{DEV}")
    total_miss = 0
    for t, x in enumerate(wl.make_tokens(spec)):
        ls.ls_predict(gl, dev_tensor(x), k, sel)
        order = sel.order()
        cache.set_priorities(sel.scores.cpu().numpy())
        ls.ls_cache_lookup(gl, sel.idx, slots, nhit)
        hits_before = cache.lookup(order)
        assert int(nhit.item()) == int(hits_before.sum())
        assert ((slots.cpu().numpy() >= 0) == hits_before).all()
        misses, victims = cache.reserve(order)
        nmiss = ls.ls_cache_reserve(gl, sel)
        assert nmiss == len(misses)
        assert snapshot(gl) == cache.resident
        total_miss += nmiss
        ls.ls_cache_lookup(gl, sel.idx, slots, nhit)
        s = slots.cpu().numpy()
        assert int(nhit.item()) == k and len(set(s.tolist())) == k and s.min() >= 0 and s.max() < C_ROWS
    st = ls.ls_cache_stats(gl)
    assert st["misses"] == total_miss == cache.misses and st["hits"] == cache.hits
    assert st["evictions"] == cache.evictions and st["resident"] == len(cache.resident)
    assert st["h2d_bytes"] == total_miss * 3 * 256 * 2
    assert 0 < total_miss < 12 * k  # the AR(1) stream re-uses neurons
    assert ls.ls_layer_status(gl) == 0
    gl.close()


def test_reserve_prefix_protect_capacity_and_evict():
    spec = ar1_spec(seed=32)
    la = wl.make_layer(spec, 0)
    C_ROWS = 64
    gl = ls.ls_layer_create(la, DEV, cache_rows=C_ROWS)
    OL = orc.OracleLayer.from_arrays(la)
    cache = orc.LogicalCache(OL.d_ff, C_ROWS)
    toks = wl.make_tokens(spec)
    sel = ls.Selection(gl.d_ff, 100, DEV)
    # fill with the first 40 ranks of token 0
    ls.ls_predict(gl, dev_tensor(toks[0]), 100, sel)
    o0 = sel.order()
    cache.set_priorities(sel.scores.cpu().numpy())
    cache.reserve(o0[:40])
    assert ls.ls_cache_reserve(gl, sel, admit_ranks=40) == 40
    assert snapshot(gl) == cache.resident == set(o0[:40].tolist())
    # token 1: 50 ranks, protecting the 10 best of token 0 -> evictions needed (40 + new > 64)
    protect = orc.mask_of(o0[:10], gl.d_ff)
    ls.ls_predict(gl, dev_tensor(toks[1]), 100, sel)
    o1 = sel.order()
    cache.set_priorities(sel.scores.cpu().numpy())
    misses, victims = cache.reserve(o1[:50], o0[:10])
    nmiss = ls.ls_cache_reserve(gl, sel, admit_ranks=50, protect_mask=dev_tensor(protect.view(np.int32)))
    assert nmiss == len(misses) and snapshot(gl) == cache.resident
    assert set(o0[:10].tolist()) <= snapshot(gl)
    # wanted + protected beyond the capacity: refused, nothing changes
    before = snapshot(gl)
    with pytest.raises(ls.LeanStreamError) as e:
        ls.ls_cache_reserve(gl, sel, admit_ranks=100, protect_mask=dev_tensor(protect.view(np.int32)))
    assert e.value.code == ls.LS_ERR_CAPACITY
    assert snapshot(gl) == before
    assert ls.ls_layer_status(gl) == ls.LS_ERR_CAPACITY
    # evict until 20 slots are free, keeping the protected ones
    ev = torch.full((C_ROWS,), -1, dtype=torch.int32, device=f"cuda:{DEV}")
    nev = torch.zeros(1, dtype=torch.int32, device=f"cuda:{DEV}")
    victims = cache.evict(20, o0[:10])
    ls.ls_cache_evict(gl, 20, dev_tensor(protect.view(np.int32)), ev, nev)
    n = int(nev.item())
    assert sorted(ev.cpu().numpy()[:n].tolist()) == victims and snapshot(gl) == cache.resident
    ls.ls_cache_evict(gl, 0)
    assert snapshot(gl) == cache.resident
    gl.close()


@pytest.mark.parametrize("K", [1, 4])
def test_cached_stack_decode_matches_oracle(K):
    """Two cached layers, AR(1) tokens: execution order (residents first), refine-driven prefetch of the next layer,
    resident sets after every step and output values, all against the oracle in replay mode."""
    spec = ar1_spec(seed=33, n_tokens=6, layers=2)
    arrays = wl.make_stack(spec, down_scale=30.0)
    OLs = [orc.OracleLayer.from_arrays(a) for a in arrays]
    C_ROWS, k = 400, 160
    GLs = [ls.ls_layer_create(a, DEV, cache_rows=C_ROWS) for a in arrays]
    plain = [ls.ls_layer_create(a, DEV) for a in arrays]
    caches = [orc.LogicalCache(1024, C_ROWS) for _ in arrays]
    sels = [ls.Selection(1024, k, DEV) for _ in range(3)]
    for x0 in wl.make_tokens(spec):
        x = dev_tensor(x0[None, :])
        ls.ls_predict(GLs[0], x, k, sels[0])
        caches[0].set_priorities(sels[0].scores.cpu().numpy())
        for n in range(2):
            last = n == 1
            gn = GLs[n] if last else GLs[n + 1]
            sel, sel_next = sels[n], sels[n + 1]
            order = sel.order()
            trace = ls.StepTrace(GLs[n], gn, K, 1, k)
            x_out = torch.empty_like(x)
            ls.ls_sparse_ffn_step(GLs[n], gn, x, x_out, sel, K, k, sel_next, trace)
            torch.cuda.synchronize()
            xt = trace.xtilde.cpu().numpy()
            res = orc.sparse_ffn_step(OLs[n], OLs[n if last else n + 1], x.cpu().numpy(), order, K, k, cache=caches[n],
                                      next_cache=None if last else caches[n + 1], xtilde_override=xt)
            assert trace.exec_idx.cpu().numpy()[:k].tolist() == res["exec_order"].tolist()
            assert snapshot(GLs[n]) == caches[n].resident
            if not last:
                assert snapshot(GLs[n + 1]) == caches[n + 1].resident
            y_ref = res["xtilde"][K] - x.cpu().numpy()
            for j in range(K + 1):
                assert_values_close(xt[j] - x.cpu().numpy(), res["xtilde"][j] - x.cpu().numpy(), scale_ref=y_ref, what=f"xt[{j}]")
            assert sel_next.order().tolist() == res["refine_orders"][K].tolist()
            # the cache changes order and residency only: same values as the all-resident layer
            x_plain = torch.empty_like(x)
            ls.ls_sparse_ffn_step(plain[n], None, x, x_plain, sel, K)
            assert_values_close((x_out - x).cpu().numpy(), (x_plain - x).cpu().numpy(), what="cached vs resident")
            x = x_out
    for n in range(2):
        st = ls.ls_cache_stats(GLs[n])
        assert (st["hits"], st["misses"], st["evictions"]) == (caches[n].hits, caches[n].misses, caches[n].evictions)
        assert ls.ls_layer_status(GLs[n]) == 0
    for g in GLs + plain:
        g.close()


def test_cached_stack_at_a_mid_size_with_eight_stages():
    """Three cached layers of a size that spans many tiles (d 1024, d_ff 8192, rank 64, k 640, 25 % cached), K = 8, an
    AR(1) stream: every step's execution order, the resident sets of both caches after every step (the refinements of the
    layer before prefetch into the next layer's cache from the copy stream), the next selection and the values."""
    spec = wl.StackSpec("cache-mid", 36, 3, 1024, 8192, True, "bf16", 64, 0.07, 4, "ar1", ar_rho=0.8)
    arrays = wl.make_stack(spec, down_scale=20.0)
    OLs = [orc.OracleLayer.from_arrays(a) for a in arrays]
    C_ROWS, k, K = 2048, 640, 8
    GLs = [ls.ls_layer_create(a, DEV, cache_rows=C_ROWS) for a in arrays]
    caches = [orc.LogicalCache(8192, C_ROWS) for _ in arrays]
    sels = [ls.Selection(8192, k, DEV) for _ in range(4)]
    n = len(GLs)
    for x0 in wl.make_tokens(spec):
        x = dev_tensor(x0[None, :])
        ls.ls_predict(GLs[0], x, k, sels[0])
        caches[0].set_priorities(sels[0].scores.cpu().numpy())
        for l in range(n):
            last = l == n - 1
            gn = GLs[l] if last else GLs[l + 1]
            sel, sel_next = sels[l], sels[l + 1]
            order = sel.order()
            trace = ls.StepTrace(GLs[l], gn, K, 1, k)
            x_out = torch.empty_like(x)
            ls.ls_sparse_ffn_step(GLs[l], gn, x, x_out, sel, K, k, sel_next, trace)
            torch.cuda.synchronize()
            xt = trace.xtilde.cpu().numpy()
            res = orc.sparse_ffn_step(OLs[l], OLs[l if last else l + 1], x.cpu().numpy(), order, K, k, cache=caches[l],
                                      next_cache=None if last else caches[l + 1], xtilde_override=xt)
            assert trace.exec_idx.cpu().numpy()[:k].tolist() == res["exec_order"].tolist()
            assert snapshot(GLs[l]) == caches[l].resident
            if not last:
                assert snapshot(GLs[l + 1]) == caches[l + 1].resident
            y_ref = res["xtilde"][K] - x.cpu().numpy()
            for j in range(K + 1):
                assert_values_close(xt[j] - x.cpu().numpy(), res["xtilde"][j] - x.cpu().numpy(), scale_ref=y_ref, what=f"xt[{j}]")
            assert sel_next.order().tolist() == res["refine_orders"][K].tolist()
            x = x_out
    for l in range(n):
        st = ls.ls_cache_stats(GLs[l])
        assert (st["hits"], st["misses"], st["evictions"]) == (caches[l].hits, caches[l].misses, caches[l].evictions)
        assert ls.ls_layer_status(GLs[l]) == 0
    for g in GLs:
        g.close()


def test_reserve_times_out_on_the_host_and_the_layer_stays_usable():
    """Failure path of the one wait the calling thread has: with the compute stream still busy with ordinary earlier work
    and a wait limit of zero, ls_cache_reserve gives up with LS_ERR_TIMEOUT and a useful message.  Nothing is lost: the
    request stays enqueued and takes effect when the stream reaches it (it COUNTS: the oracle's cache makes the same
    reserve), the next call works, and the resident set equals the oracle's."""
    spec = ar1_spec(seed=35)
    la = wl.make_layer(spec, 0)
    C_ROWS, k = 300, 160
    gl = ls.ls_layer_create(la, DEV, cache_rows=C_ROWS)
    cache = orc.LogicalCache(1024, C_ROWS)
    sel = ls.Selection(gl.d_ff, k, DEV)
    toks = wl.make_tokens(spec)
    try:
        ls.ls_predict(gl, dev_tensor(toks[0]), k, sel)
        cache.set_priorities(sel.scores.cpu().numpy())
        order = sel.order()
        torch.cuda.synchronize()
        ls.ls_set_option(ls.LS_OPT_HOST_WAIT_MS, 0)
        # ordinary work that keeps the stream busy for a moment (a few large matrix products), then the reserve behind it
        a = torch.randn(8192, 8192, device=f"cuda:{DEV}")
        for _ in range(20):
            a = (a @ a).clamp_(-1, 1)
        with pytest.raises(ls.LeanStreamError) as e:
            ls.ls_cache_reserve(gl, sel)
        assert e.value.code == ls.LS_ERR_TIMEOUT and "timed out" in str(e.value)
    finally:
        ls.ls_set_option(ls.LS_OPT_HOST_WAIT_MS, 30000)
    torch.cuda.synchronize()
    misses, _ = cache.reserve(order)  # the request that timed out on the host did run
    assert snapshot(gl) == cache.resident
    st = ls.ls_cache_stats(gl)
    assert st["misses"] == len(misses) == cache.misses
    ls.ls_predict(gl, dev_tensor(toks[1]), k, sel)
    cache.set_priorities(sel.scores.cpu().numpy())
    m2, _ = cache.reserve(sel.order())
    assert ls.ls_cache_reserve(gl, sel) == len(m2)
    assert snapshot(gl) == cache.resident and ls.ls_layer_status(gl) == 0
    gl.close()
