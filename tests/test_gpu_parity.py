"""Parity of the CUDA library (through the C ABI) against the CPU oracle, element by element, on seeded inputs."""
import copy

import numpy as np
import pytest
import torch

from oracle import leanstream_oracle as orc
from paper_2609_03079_b200 import binding as ls
from paper_2609_03079_b200 import workload as wl
from tests.helpers import assert_values_close, check_selection, check_survive, mask_to_set

pytestmark = pytest.mark.gpu
DEV = 0


@pytest.fixture(autouse=True, params=[1, 0], ids=["fused", "staged"])
def kernel_path(request):
    """Every test runs on both implementations of the step: the fused per-layer kernel and the stage-by-stage kernels."""
    ls.ls_set_option(ls.LS_OPT_FUSED, request.param)
    yield request.param
    ls.ls_set_option(ls.LS_OPT_FUSED, 1)


def dev_tensor(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda(DEV)


def custom_arrays(seed, d, F, r, gated=True, wdtype="bf16", activity=0.2, down_scale=1.0):
    spec = wl.StackSpec("custom", seed, 1, d, F, gated, wdtype, r, activity, 4, "iid")
    return spec, wl.make_layer(spec, 0, down_scale=down_scale)


def run_step_and_compare(gl, gn, OL, ON, x_np, k, K, k_next, stats, batch_order=None):
    """One ls_sparse_ffn_step against the oracle in replay mode; returns (x_out, next order) from the GPU."""
    X = np.atleast_2d(x_np).astype(np.float32)
    B = X.shape[0]
    x = dev_tensor(X)
    sel = ls.Selection(gl.d_ff, min(B * k, gl.d_ff), DEV)
    ls.ls_predict(gl, x, k, sel)
    order = sel.order()
    o_ref, prio_ref = orc.select_batch(OL, X, k)
    if B == 1:
        check_selection(order, orc.predictor_scores(OL, X[0]), k, stats)
    else:
        assert order.tolist() == o_ref.tolist()
    np.testing.assert_allclose(sel.scores.cpu().numpy(), prio_ref, rtol=1e-11, atol=1e-12)
    assert mask_to_set(sel.mask_np(), gl.d_ff) == set(order.tolist())

    sel_next = ls.Selection(gn.d_ff, min(B * k_next, gn.d_ff), DEV)
    trace = ls.StepTrace(gl, gn, K, B, sel.cap)
    x_out = torch.empty_like(x)
    ls.ls_sparse_ffn_step(gl, gn, x, x_out, sel, K, k_next, sel_next, trace)
    torch.cuda.synchronize()
    assert ls.ls_layer_status(gl) == 0 and ls.ls_layer_status(gn) == 0

    xt_gpu = trace.xtilde.cpu().numpy()  # [K+1, B, d]
    res = orc.sparse_ffn_step(OL, ON, X, order, K, k_next, xtilde_override=xt_gpu)
    # values: every partial feature's increment over x, and the final output
    y_ref = res["xtilde"][K] - X
    for j in range(K + 1):
        assert_values_close(xt_gpu[j] - X, res["xtilde"][j] - X, scale_ref=y_ref, what=f"xtilde[{j}]")
    np.testing.assert_array_equal(x_out.cpu().numpy(), xt_gpu[K])
    assert trace.exec_idx.cpu().numpy()[: len(order)].tolist() == order.tolist()
    # refined sets for the next layer, from the GPU's own feature bits: bit-exact
    masks = trace.refine_masks.cpu().numpy().view(np.uint32)
    counts = trace.refine_counts.cpu().numpy()
    for j in range(K + 1):
        ref_order = res["refine_orders"][j]
        assert counts[j] == len(ref_order)
        got = mask_to_set(masks[j], gn.d_ff)
        if B == 1:
            s = orc.predictor_scores(ON, xt_gpu[j, 0])
            gpu_sorted = np.asarray(sorted(got, key=lambda i: (-orc._canonical(s)[i], i)), dtype=np.int64)
            check_selection(gpu_sorted, s, k_next, stats)
        else:
            assert got == set(ref_order.tolist())
    nxt_order = sel_next.order()
    if B == 1:
        check_selection(nxt_order, orc.predictor_scores(ON, xt_gpu[K, 0]), k_next, stats)
    else:
        assert nxt_order.tolist() == res["refine_orders"][K].tolist()
    if B == 1:
        check_survive(mask_to_set(trace.survive_mask.cpu().numpy().view(np.uint32), gl.d_ff), OL, X[0], order)
    return x_out.cpu().numpy(), nxt_order


@pytest.fixture(scope="module")
def tiny():
    spec = wl.SPECS["tiny"]
    la = wl.make_layer(spec, 0)
    gl = ls.ls_layer_create(la, DEV, max_batch=4)
    yield spec, la, orc.OracleLayer.from_arrays(la), gl, wl.make_tokens(spec)
    gl.close()


def test_predict_tiny_bit_exact(tiny):
    spec, la, OL, gl, toks = tiny
    stats = {}
    sel = ls.Selection(gl.d_ff, spec.k, DEV)
    for x in toks:
        ls.ls_predict(gl, dev_tensor(x), spec.k, sel)
        s_ref = orc.predictor_scores(OL, x)
        check_selection(sel.order(), s_ref, spec.k, stats)
        np.testing.assert_allclose(sel.scores.cpu().numpy(), s_ref, rtol=1e-12, atol=1e-13)
        assert sel.mask_np().tolist() == orc.mask_of(sel.order(), gl.d_ff).tolist()
    assert stats.get("band", 0) == 0 and stats["exact"] == len(toks)
    # selection kernels are deterministic: same input, same bits
    a = sel.idx.clone()
    ls.ls_predict(gl, dev_tensor(toks[-1]), spec.k, sel)
    assert torch.equal(a, sel.idx)


@pytest.mark.parametrize("k", [0, 1, 31, 1024])
def test_predict_k_edges(tiny, k):
    spec, la, OL, gl, toks = tiny
    sel = ls.Selection(gl.d_ff, max(k, 1), DEV)
    ls.ls_predict(gl, dev_tensor(toks[0]), k, sel)
    assert sel.order().tolist() == orc.topk_order(orc.predictor_scores(OL, toks[0]), k).tolist()


def test_predict_exact_ties_lower_index_first(tiny):
    spec, la, OL, gl, toks = tiny
    pairs = [(5, 700), (123, 124), (1000, 3)]
    lt = wl.tied_duplicate_layer(la, pairs)
    gt = ls.ls_layer_create(lt, DEV)
    OT = orc.OracleLayer.from_arrays(lt)
    sel = ls.Selection(gt.d_ff, gt.d_ff, DEV)
    for x in toks[:4]:
        ls.ls_predict(gt, dev_tensor(x), gt.d_ff, sel)
        s = sel.scores.cpu().numpy()
        order = sel.order().tolist()
        for a, b in pairs:
            assert s[a] == s[b]
            lo, hi = min(a, b), max(a, b)
            assert order.index(lo) + 1 == order.index(hi)
        assert order == orc.topk_order(orc.predictor_scores(OT, x), gt.d_ff).tolist()
    gt.close()


def test_refined_sets_with_exact_ties_in_the_next_layer(tiny):
    """The next layer has duplicated predictor columns: its refined order must still put the lower index first."""
    spec, la, OL, gl, toks = tiny
    pairs = [(5, 700), (123, 124), (1000, 3), (64, 65), (8, 1016)]
    lt = wl.tied_duplicate_layer(la, pairs)
    gt = ls.ls_layer_create(lt, DEV)
    OT = orc.OracleLayer.from_arrays(lt)
    stats = {}
    for x in toks[:6]:
        run_step_and_compare(gl, gt, OL, OT, x, spec.k, 8, 1024, stats)  # k_next = d_ff: the full order is compared
    assert stats.get("band", 0) == 0
    gt.close()


def test_predict_degenerate_all_equal_scores():
    """Zero predictor and constant bias: every score equal, so the order is the index order."""
    spec, la = custom_arrays(11, 64, 300, 8)
    la.pred_b[:] = 0
    la.pred_c[:] = 0.25
    gl = ls.ls_layer_create(la, DEV)
    sel = ls.Selection(300, 300, DEV)
    ls.ls_predict(gl, dev_tensor(wl.make_tokens(spec)[0]), 77, sel)
    assert sel.order().tolist() == list(range(77))
    gl.close()


@pytest.mark.parametrize("K", [1, 3, 8])
def test_step_tiny_against_oracle(tiny, K):
    spec, la, OL, gl, toks = tiny
    stats = {}
    for x in toks[: (16 if K == 8 else 4)]:
        run_step_and_compare(gl, gl, OL, OL, x, spec.k, K, spec.k, stats)
    assert stats.get("band", 0) == 0


def test_step_k_equals_dff_is_dense(tiny):
    spec, la, OL, gl, toks = tiny
    x = dev_tensor(toks[1])
    sel = ls.Selection(gl.d_ff, gl.d_ff, DEV)
    ls.ls_predict(gl, x, gl.d_ff, sel)
    x_out = torch.empty_like(x)
    ls.ls_sparse_ffn_step(gl, None, x, x_out, sel, 4)
    y = (x_out - x).cpu().numpy().astype(np.float64)
    assert_values_close(y, orc.dense_ffn(OL, toks[1]), what="dense")


def test_step_in_place_and_more_chunks_than_neurons(tiny):
    spec, la, OL, gl, toks = tiny
    x = dev_tensor(toks[2])
    sel = ls.Selection(gl.d_ff, 5, DEV)
    ls.ls_predict(gl, x, 5, sel)
    ref = orc.sparse_ffn_step(OL, None, toks[2], sel.order(), 9)
    xin = x.clone()
    ls.ls_sparse_ffn_step(gl, None, xin, xin, sel, 9)  # K > k: empty stages; x_out aliases x
    assert_values_close((xin - x).cpu().numpy(), ref["y"][0], what="in-place")
    # empty selection leaves x unchanged
    ls.ls_predict(gl, x, 0, sel)
    out = torch.empty_like(x)
    ls.ls_sparse_ffn_step(gl, None, x, out, sel, 2)
    assert torch.equal(out, x)


def test_ragged_shapes_and_tail_stage():
    """d_model not a multiple of the 256-lane tile, d_ff not a multiple of 32, rank 40, k not divisible by K."""
    spec, la = custom_arrays(21, 264, 1000, 40, activity=0.25)
    gl = ls.ls_layer_create(la, DEV)
    OL = orc.OracleLayer.from_arrays(la)
    stats = {}
    for x in wl.make_tokens(spec):
        run_step_and_compare(gl, gl, OL, OL, x, 77, 5, 91, stats)
    gl.close()


def test_fp16_non_gated_layer():
    spec, la = custom_arrays(22, 512, 2048, 64, gated=False, wdtype="fp16", activity=0.1)
    la.b_down = (np.arange(512, dtype=np.float32) % 7 - 3) * 1e-3
    gl = ls.ls_layer_create(la, DEV)
    OL = orc.OracleLayer.from_arrays(la)
    stats = {}
    for x in wl.make_tokens(spec)[:2]:
        run_step_and_compare(gl, gl, OL, OL, x, 224, 4, 224, stats)
    gl.close()


def test_fp16_gated_layer_on_the_tensor_core_dot_products():
    """fp16 weights, gated, d a multiple of 16: the whole-token kernel's gate and up dot products run as fp16 MMAs on x cut
    into three fp16 terms (scaled by 2^11 per term); tokens of very different magnitudes exercise the scaling."""
    spec, la = custom_arrays(24, 512, 2048, 64, gated=True, wdtype="fp16", activity=0.15)
    gl = ls.ls_layer_create(la, DEV)
    OL = orc.OracleLayer.from_arrays(la)
    stats = {}
    toks = wl.make_tokens(spec)
    for x, scale in zip(toks[:3], (1.0, 1e-3, 300.0)):
        run_step_and_compare(gl, gl, OL, OL, (x * scale).astype(np.float32), 320, 4, 320, stats)
    gl.close()


def test_feature_wider_than_one_pass_of_the_block():
    """d = 6144 > 4096 columns: a thread owns more than one group of eight output columns, so the partial output is
    accumulated in the CTA's global row instead of registers; rows of 12 KB, several ring batches."""
    spec, la = custom_arrays(25, 6144, 2048, 64, activity=0.2)
    gl = ls.ls_layer_create(la, DEV)
    OL = orc.OracleLayer.from_arrays(la)
    stats = {}
    for x in wl.make_tokens(spec)[:2]:
        run_step_and_compare(gl, gl, OL, OL, x, 448, 8, 448, stats)
    gl.close()


def test_batch_union(tiny):
    spec, la, OL, gl, toks = tiny
    stats = {}
    run_step_and_compare(gl, gl, OL, OL, toks[:4], 96, 4, 96, stats)
    # a batch of copies behaves like batch 1
    X = np.stack([toks[5]] * 3)
    sel = ls.Selection(gl.d_ff, 3 * 96, DEV)
    ls.ls_predict(gl, dev_tensor(X), 96, sel)
    assert sel.order().tolist() == orc.topk_order(orc.predictor_scores(OL, toks[5]), 96).tolist()


def test_tiny4_stack_with_moving_refinement():
    spec = wl.SPECS["tiny4"]
    arrays = wl.make_stack(spec, down_scale=50.0)
    OLs = [orc.OracleLayer.from_arrays(a) for a in arrays]
    GLs = [ls.ls_layer_create(a, DEV) for a in arrays]
    stats = {}
    moved = 0
    for x0 in wl.make_tokens(spec)[:3]:
        x = x0
        for n in range(4):
            nn = min(n + 1, 3)
            x_new, nxt_order = run_step_and_compare(GLs[n], GLs[nn], OLs[n], OLs[nn], x, spec.k, 4, spec.k, stats)
            first = orc.topk_order(orc.predictor_scores(OLs[nn], x), spec.k)
            moved += len(set(first.tolist()) ^ set(nxt_order.tolist()))
            x = x_new[0]
    assert moved > 0 and stats.get("band", 0) == 0
    for g in GLs:
        g.close()


def test_argument_errors(tiny):
    spec, la, OL, gl, toks = tiny
    x = dev_tensor(toks[0])
    sel = ls.Selection(gl.d_ff, 10, DEV)
    with pytest.raises(ls.LeanStreamError) as e:
        ls.ls_predict(gl, x, 11, sel)  # cap too small
    assert e.value.code == ls.LS_ERR_INVALID
    with pytest.raises(ls.LeanStreamError):
        ls.ls_predict(gl, x, gl.d_ff + 1, sel)
    with pytest.raises(ls.LeanStreamError) as e:
        ls.ls_cache_lookup(gl, sel.idx, sel.idx.clone())
    assert e.value.code == ls.LS_ERR_STATE
    bad = copy.copy(la)
    bad.d_model = 250
    with pytest.raises(ls.LeanStreamError):
        ls.ls_layer_create(bad, DEV)
    # an out-of-range neuron index is skipped and reported, never dereferenced
    ls.ls_predict(gl, x, 10, sel)
    sel.idx[3] = 5000
    out = torch.empty_like(x)
    ls.ls_sparse_ffn_step(gl, None, x, out, sel, 2)
    assert ls.ls_layer_status(gl) == ls.LS_ERR_INVALID
    assert ls.ls_layer_status(gl) == 0


def test_llama7b_shaped_layer_full_size():
    """One layer at the benchmark's shape (d 4096, d_ff 11008, rank 256, k 1728, K 8), full comparison on 2 tokens."""
    spec = wl.SPECS["llama2-7b"]
    la = wl.make_layer(spec, 0, svd_device="cuda")
    lb = wl.make_layer(spec, 1, svd_device="cuda")
    ga, gb = ls.ls_layer_create(la, DEV), ls.ls_layer_create(lb, DEV)
    OA, OB = orc.OracleLayer.from_arrays(la), orc.OracleLayer.from_arrays(lb)
    stats = {}
    for x in wl.make_tokens(spec, 2):
        run_step_and_compare(ga, gb, OA, OB, x, spec.k, 8, spec.k, stats)
    assert stats.get("band", 0) == 0
    ga.close()
    gb.close()


def test_llama7b_shaped_layer_wide_selection():
    """Benchmark-shaped layer pair with k = 6016 (more members than the selection keeps in shared memory: the grouped
    members go through the global scratch) and with the intermediate refined sets traced."""
    spec = wl.SPECS["llama2-7b"]
    la = wl.make_layer(spec, 0, svd_device="cuda")
    lb = wl.make_layer(spec, 1, svd_device="cuda")
    ga, gb = ls.ls_layer_create(la, DEV), ls.ls_layer_create(lb, DEV)
    OA, OB = orc.OracleLayer.from_arrays(la), orc.OracleLayer.from_arrays(lb)
    stats = {}
    x = wl.make_tokens(spec, 1)[0]
    run_step_and_compare(ga, gb, OA, OB, x, 6016, 3, 6016, stats)
    assert stats.get("band", 0) == 0
    ga.close()
    gb.close()


@pytest.mark.parametrize("gated", [True, False])
def test_silu_layers(gated):
    """The activation Eq. 1 prints (SiLU): no exact zeros, so every selected neuron contributes its up and down rows;
    values against the oracle's SiLU branch, sets bit-exact as always, on ragged shapes."""
    spec, la = custom_arrays(23, 264, 1000, 40, gated=gated, wdtype="bf16" if gated else "fp16")
    la.act = "silu"
    if not gated:
        la.b_down = (0.01 * np.arange(264, dtype=np.float32) - 1.0)
    OL = orc.OracleLayer.from_arrays(la)
    assert OL.act == orc.SILU
    gl = ls.ls_layer_create(la, DEV)
    stats = {}
    for x in wl.make_tokens(spec):
        run_step_and_compare(gl, gl, OL, OL, x, 77, 5, 130, stats)
    assert stats.get("band", 0) == 0
    gl.close()
