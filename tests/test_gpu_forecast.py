"""End-to-end parity of the CUDA decoder with the oracle on the five workloads (and small
ragged variants), through the C ABI, plus properties that hold at any size."""
import os

import numpy as np
import pytest
import torch

import tests.parity as parity
from tests.gpu_common import make_decoder, series_on_device
from oracle import tsfm_oracle as orc
from tsfm_inputs import Arch, WORKLOADS, workload

pytestmark = pytest.mark.gpu


def check_stats(st, B, T, K):
    d = st.as_dict()
    assert d["device_status"] == 0
    assert d["patches_committed"] == B * T
    assert 1 <= d["rounds"] <= T
    assert d["proposals_accepted"] <= d["proposals_tested"] <= d["proposals_drafted"]
    n_rounds = sum(d["L_hist"])
    assert d["proposals_drafted"] == K * n_rounds
    assert sum(d["L_hist"][K + 2:]) == 0 and d["L_hist"][0] == 0
    assert sum(l * c for l, c in enumerate(d["L_hist"])) == n_rounds + d["proposals_accepted"]
    tested, acc = np.array(d["tested_by_pos"][:K], float), np.array(d["accepted_by_pos"][:K], float)
    assert tested[0] == n_rounds and np.all(tested[1:] == acc[:-1])
    # the capped-geometric identity on the run's own counts: mean(L) = sum_l prod_{i<l} a_i
    rate = np.divide(acc, tested, out=np.zeros(K), where=tested > 0)
    mean_L = sum(l * c for l, c in enumerate(d["L_hist"])) / n_rounds
    assert mean_L == pytest.approx(sum(np.prod(rate[:l]) for l in range(K + 1)), rel=1e-9)
    return d


def run_and_compare(wl, K, tau, seed, ids, backend=0, batch=None, H=None, exec_mode=0):
    H = H or wl.horizon
    B = batch or wl.batch
    ids = list(ids)
    dec, tw, dw = make_decoder(wl, backend=backend, max_K=max(K, wl.K), batch=B, exec_mode=exec_mode)
    s, ctx = series_on_device(wl, B)
    out, st = dec.forecast(ctx, H, K, tau, seed)
    T = -(-H // wl.patch_len)
    d = check_stats(st, B, T, K)
    nacc, ell, logu = dec.last_trace(B, K)
    assert nacc.shape[0] == d["rounds"]
    # the decoder's near-margin counter is the count over its own trace
    assert d["near_margin_decisions"] == parity.gpu_near_margin_total(nacc, ell, logu, K, parity.MARGIN[wl.dtype])
    ref, st0 = dec.target_only(ctx, H)
    got = out.cpu().numpy()
    tgt_only = ref.cpu().numpy()
    dec.close()
    tm, dm = parity.oracle_models(wl, tw, dw)
    res = parity.compare_forecast(wl, tm, dm, s, H, K, tau, seed, got, nacc, ids, gpu_ell=ell, gpu_logu=logu)
    want_t = parity.oracle_target_only(tm, s, wl.ctx_len, H, ids)
    kind, tol = parity.VALUE_TOL[wl.dtype]
    each = parity.per_series_errors(kind, tgt_only[ids], want_t)
    res["target_only_error"] = float(each.max())
    assert each.max() <= tol, f"target-only, series {ids[int(each.argmax())]}: {kind} error {each.max():.4g} > {tol}"
    res["stats"] = d
    print(wl.name, K, tau, {k: v for k, v in res.items() if k != "stats"},
          "acc", d["proposals_accepted"], "/", d["proposals_tested"], "rounds", d["rounds"])
    return res


def spread(B, n):
    """n series ids spread over a batch of B (first, last and evenly spaced ones between)."""
    return sorted(set(int(round(i * (B - 1) / (n - 1))) for i in range(n)))


EXEC = pytest.mark.parametrize("exec_mode", [1, 0], ids=["stream", "graph"])


@EXEC
def test_c0_full(exec_mode):
    wl = workload("C0")
    run_and_compare(wl, wl.K, wl.tau, wl.forecast_seed, range(wl.batch), exec_mode=exec_mode)


@EXEC
@pytest.mark.parametrize("K,tau,H", [(1, 1.0, 384), (3, 2.0, 400), (4, 4.0, 96 * 7 + 5)])
def test_c0_shape_ragged_batch_fp32(K, tau, H, exec_mode):
    """C0's models on a ragged batch: several series, acceptance in the middle range, truncated last patch."""
    wl = workload("C0", batch=6, series_recipe="c1", horizon=H)
    run_and_compare(wl, K, tau, 7, range(6), exec_mode=exec_mode)


@pytest.mark.parametrize("backend,exec_mode", [(1, 1), (0, 1), (0, 0)],
                         ids=["simt-stream", "tcgen05-stream", "tcgen05-graph"])
@pytest.mark.parametrize("tau", [0.5, 1.0, 2.0])
def test_c1_full(tau, backend, exec_mode):
    wl = workload("C1")
    run_and_compare(wl, wl.K, tau, wl.forecast_seed, range(wl.batch), backend=backend, exec_mode=exec_mode)


def test_c1_with_a_draft_that_tracks_its_target():
    """The regime the paper reports (acceptance 49-97 %): C1's layer-skip pair with the target's layers
    beyond the draft's depth damped to a tenth, 15 patches to commit.  Most rounds yield K + 1."""
    wl = workload("C1", late_layer_scale=0.1, horizon=1440)
    res = run_and_compare(wl, wl.K, 1.0, wl.forecast_seed, range(0, wl.batch, 2))
    d = res["stats"]
    assert d["proposals_accepted"] / d["proposals_tested"] > 0.9
    assert d["rounds"] <= 6


def test_graph_and_stream_execution_give_identical_forecasts_and_traces():
    """The captured graph (device-side WHILE over rounds) replays exactly what the stream path
    launches: same kernels, same arguments -- so forecasts, decisions and counters are identical,
    also when one handle replays its graph with other seeds, temperatures and block sizes."""
    wl = workload("C0", batch=5, series_recipe="c1")          # fp32 path: bit-reproducible
    s, ctx = series_on_device(wl)
    decs = [make_decoder(wl, max_K=4, exec_mode=m)[0] for m in (1, 0)]
    for K, tau, seed in [(2, 1.0, 3), (2, 2.5, 4), (4, 2.5, 4), (1, 0.7, 9), (2, 1.0, 3)]:
        res = []
        for dec in decs:
            out, st = dec.forecast(ctx, wl.horizon, K, tau, seed)
            nacc, ell, logu = dec.last_trace(wl.batch, K)
            d = st.as_dict()
            res.append((out.cpu().numpy(), nacc, ell, logu,
                        {k: d[k] for k in ("rounds", "proposals_tested", "proposals_accepted", "L_hist")}))
        for a, b in zip(res[0][:4], res[1][:4]):
            np.testing.assert_array_equal(a, b)
        assert res[0][4] == res[1][4]
        assert res[1][4]["rounds"] == res[1][1].shape[0]
    ref = [dec.target_only(ctx, wl.horizon)[0].cpu().numpy() for dec in decs]
    np.testing.assert_array_equal(ref[0], ref[1])
    for dec in decs:
        dec.close()


@pytest.mark.parametrize("name", ["fp32", "bf16-small-M", "bf16-many-rows"])
def test_compaction_of_finished_series_changes_nothing(name):
    """Rounds run over the unfinished series only (slots of a compacted batch); with the flag that
    switches this off every round runs over all series.  Series never interact, so forecasts,
    decisions and counters must be the same -- bit for bit: a row's arithmetic does not depend on
    where in the batch it sits."""
    import paper_2511_18191_b200 as tsfm
    if name == "fp32":
        wl, K, tau = workload("C0", batch=7, series_recipe="c1", horizon=96 * 9 + 5), 3, 2.0
    elif name == "bf16-small-M":
        wl, K, tau = workload("C1", batch=12, horizon=96 * 10), 4, 2.0
    else:      # enough rows for the large-tile contractions and the shared-load embedding / head kernels
        wl, K, tau = workload("C3", draft_eps=1e-1, horizon=96 * 9, target=Arch(2, 256, 4, 512),
                              draft=Arch(2, 256, 4, 512)), 4, 0.3
    s, ctx = series_on_device(wl)
    res = []
    for mode in (tsfm.TSFM_EXEC_GRAPH, tsfm.TSFM_EXEC_GRAPH | tsfm.TSFM_EXEC_NO_COMPACT,
                 tsfm.TSFM_EXEC_STREAM, tsfm.TSFM_EXEC_STREAM | tsfm.TSFM_EXEC_NO_COMPACT):
        dec = make_decoder(wl, max_K=K, exec_mode=mode)[0]
        out, st = dec.forecast(ctx, wl.horizon, K, tau, 5)
        nacc, ell, logu = dec.last_trace(wl.batch, K)
        d = st.as_dict()
        res.append((out.cpu().numpy(), nacc, {k: d[k] for k in ("rounds", "proposals_tested", "proposals_accepted", "L_hist")}))
        dec.close()
    finished_at = (res[0][1] >= 0).sum(axis=0)                  # rounds each series took part in
    assert finished_at.min() < finished_at.max(), "the case must desynchronise the batch"
    for other in res[1:]:
        np.testing.assert_array_equal(res[0][1], other[1])
        np.testing.assert_array_equal(res[0][0], other[0])
        assert res[0][2] == other[2]


BOUNDS_CASES = {
    "fp32-ragged": lambda: (workload("C0", batch=6, series_recipe="c1", horizon=96 * 7 + 5), 4, 4.0),
    "bf16-small-M": lambda: (workload("C1", batch=12, horizon=96 * 10), 4, 2.0),
    "bf16-K-beyond-a-tile": lambda: (workload("C1", batch=4, horizon=96 * 6), 20, 2.0),
    "bf16-long-rows": lambda: (workload("C4", batch=3, horizon=32 * 11 + 7, target=Arch(2, 256, 4, 512),
                                        draft=Arch(1, 128, 2, 256)), 8, 1.0),
    "bf16-many-rows": lambda: (workload("C3", draft_eps=1e-1, horizon=96 * 5, target=Arch(2, 256, 4, 512),
                                        draft=Arch(2, 256, 4, 512)), 4, 0.3),
    "bf16-point-tokens": lambda: (workload("C5", batch=5, horizon=64 * 3 + 9), 3, 1.0),
}


@pytest.mark.parametrize("name", sorted(BOUNDS_CASES))
def test_bounds_checking_mode_finds_no_write_outside_any_buffer(name):
    """In bounds-checking mode every buffer has guard bytes behind it and every (layer, series, head)
    block of the KV caches and every series' history a spare last token; a kernel inspects them after
    each call.  Representative forecasts (ragged positions, full rollbacks, K + 1 beyond one query
    tile, rows of 300 tokens, 1024 series, point tokens), in both execution modes, leave them intact,
    and give the same numbers as the ordinary mode."""
    import paper_2511_18191_b200 as tsfm
    wl, K, tau = BOUNDS_CASES[name]()
    s, ctx = series_on_device(wl)
    outs = []
    for mode in (tsfm.TSFM_EXEC_GRAPH, tsfm.TSFM_EXEC_GRAPH | tsfm.TSFM_EXEC_CHECK_BOUNDS,
                 tsfm.TSFM_EXEC_STREAM | tsfm.TSFM_EXEC_CHECK_BOUNDS):
        dec = make_decoder(wl, max_K=K, exec_mode=mode)[0]
        checked = bool(mode & tsfm.TSFM_EXEC_CHECK_BOUNDS) or os.environ.get("TSFM_TEST_CHECK_BOUNDS") == "1"
        assert (tsfm.tsfm_spec_debug_guard(dec.h) > 20) == checked
        out, st = dec.forecast(ctx, wl.horizon, K, tau, 3)           # raises if a guard is damaged
        assert st.device_status == 0
        ref, st_t = dec.target_only(ctx, wl.horizon)
        dro, st_d = dec.draft_only(ctx, wl.horizon)
        assert st_t.device_status == 0 and st_d.device_status == 0
        outs.append((out.cpu().numpy(), ref.cpu().numpy(), dro.cpu().numpy()))
        dec.close()
    for other in outs[1:]:
        for a, b in zip(outs[0], other):
            np.testing.assert_array_equal(a, b)


def test_a_damaged_guard_is_reported_by_name_and_the_handle_recovers():
    """The checker itself: one byte of a guard region overwritten from the host (a write inside the
    library's own allocation) makes the next call fail with the buffer's name; restored, calls succeed."""
    import paper_2511_18191_b200 as tsfm
    wl = workload("C0", batch=2, series_recipe="c1")
    dec = make_decoder(wl, exec_mode=tsfm.TSFM_EXEC_GRAPH | tsfm.TSFM_EXEC_CHECK_BOUNDS)[0]
    s, ctx = series_on_device(wl)
    n = tsfm.tsfm_spec_debug_guard(dec.h)
    dec.forecast(ctx, wl.horizon, wl.K, 1.0, 1)
    for region in (0, n // 2, n - 1):
        tsfm.tsfm_spec_debug_guard(dec.h, region, damage=True)
        with pytest.raises(tsfm.TsfmError) as e:
            dec.forecast(ctx, wl.horizon, wl.K, 1.0, 1)
        assert e.value.code == tsfm.TSFM_ERR_INTERNAL and f"guard region {region})" in str(e.value)
        tsfm.tsfm_spec_debug_guard(dec.h, region, damage=False)
        dec.forecast(ctx, wl.horizon, wl.K, 1.0, 1)
    dec.close()


def test_launch_counter_counts_replayed_rounds():
    import paper_2511_18191_b200 as tsfm
    wl = workload("C0", batch=3, series_recipe="c1")
    s, ctx = series_on_device(wl)
    counts = []
    for mode in (1, 0):
        dec, _, _ = make_decoder(wl, exec_mode=mode)
        dec.forecast(ctx, wl.horizon, wl.K, 2.0, 1)            # warm-up (captures the graph in graph mode)
        n0 = tsfm.tsfm_launch_count()
        dec.forecast(ctx, wl.horizon, wl.K, 2.0, 1, stats=False)
        dec.target_only(ctx, wl.horizon, stats=False)
        counts.append(tsfm.tsfm_launch_count() - n0)
        dec.close()
        assert tsfm.tsfm_launch_count() - n0 == counts[-1]      # survives the handle
    assert counts[0] == counts[1] and counts[0] > 0


def test_c2_sixteen_series():
    wl = workload("C2")
    res = run_and_compare(wl, wl.K, wl.tau, wl.forecast_seed, spread(wl.batch, 16))
    assert res["series"] == 16


@pytest.mark.parametrize("K", [1, 2, 4, 8])            # (the upper decorator varies fastest: weights are reused)
@pytest.mark.parametrize("eps", [0.0, 1e-3, 1e-2, 1e-1])
def test_c3_whole_sweep(K, eps):
    """Every cell of the K x eps grid, 16 series each.  eps = 0 is a draft that is the target:
    everything is accepted and every round yields K + 1.  With this build's perturbation recipe
    (eps x the tensor's standard deviation) eps = 1e-1 still accepts about nine proposals in ten at
    tau = 1; the low end of the acceptance range is reached through tau (next test)."""
    wl = workload("C3", draft_eps=eps)
    res = run_and_compare(wl, K, wl.tau, wl.forecast_seed, spread(wl.batch, 16))
    d = res["stats"]
    if eps == 0.0:                       # draft == target: everything accepted, every round yields K+1
        assert d["proposals_accepted"] == d["proposals_tested"]
        assert d["rounds"] == -(-wl.n_patches // (K + 1))
    else:
        assert d["proposals_accepted"] < d["proposals_tested"] or eps < 1e-1


@pytest.mark.parametrize("tau,lo,hi", [(0.3, 0.05, 0.9), (0.1, 0.0, 0.1)])
def test_c3_low_acceptance_end(tau, lo, hi):
    """The most perturbed draft of the sweep at small acceptance temperatures: ragged per-series
    acceptance in the middle of the range, then hardly any (every round yields one patch)."""
    wl = workload("C3", draft_eps=1e-1)
    res = run_and_compare(wl, 4, tau, wl.forecast_seed, spread(wl.batch, 16))
    d = res["stats"]
    assert lo <= d["proposals_accepted"] / d["proposals_tested"] <= hi


def test_c4_sixteen_series():
    wl = workload("C4")
    res = run_and_compare(wl, wl.K, wl.tau, wl.forecast_seed, spread(wl.batch, 16))
    assert res["series"] == 16


def test_c5_point_tokens_every_series():
    """The point-token family: input tokens of one step, a 64-step head, so a committed patch is 64
    tokens and the verification pass over [pending, x_1..x_K] is read at every 64th token (the
    prefix boundaries N - 1 + i P / P_in)."""
    wl = workload("C5")
    for mode in (1, 0):
        res = run_and_compare(wl, wl.K, wl.tau, wl.forecast_seed, range(wl.batch), exec_mode=mode)
    assert res["series"] == wl.batch


@pytest.mark.parametrize("P,P_in,K,H", [(16, 4, 3, 16 * 5 + 3), (32, 16, 2, 32 * 4), (16, 1, 4, 16 * 3 + 1)])
def test_short_input_tokens_fp32(P, P_in, K, H):
    """Input tokens shorter than the patch on the fp32 path (several tokens per patch, with and
    without the 16-byte embedding loads), ragged batch, truncated last patch."""
    wl = workload("C0", batch=5, series_recipe="c1", patch_len=P, patch_in=P_in, ctx_len=P * 6, horizon=H)
    for mode in (1, 0):
        run_and_compare(wl, K, 2.0, 13, range(5), exec_mode=mode)


@pytest.mark.parametrize("target,draft", [
    (Arch(2, 256, 2, 512), Arch(1, 64, 2, 128)),      # head sizes 128 and 32
    (Arch(2, 256, 4, 512), Arch(1, 128, 2, 256)),     # head size 64
])
def test_long_rows_small_models_bf16(target, draft):
    """C4's row lengths (256 context tokens, K = 8) on small models: the running-softmax attention
    with the keys of a row dealt out over four warps, for every head size, ragged batch of 3."""
    wl = workload("C4", batch=3, horizon=32 * 11 + 7, target=target, draft=draft)
    run_and_compare(wl, wl.K, wl.tau, wl.forecast_seed, [0, 1, 2])
    run_and_compare(wl, 3, 2.0, 3, [0, 1, 2], exec_mode=1)


def test_long_rows_fp32_keys_split_over_a_cluster():
    """fp32 caches of 200+ rows: the keys of a (series, head) are split over a cluster of four CTAs
    whose partial softmax results are merged through distributed shared memory, in prefill (13
    query tiles), verification (4 queries) and one-token steps alike."""
    wl = workload("C0", batch=2, series_recipe="c1", ctx_len=96 * 200, horizon=96 * 4 + 10)
    for mode in (1, 0):
        run_and_compare(wl, 3, 2.0, 4, [0, 1], exec_mode=mode)


def test_block_size_beyond_one_query_tile_bf16():
    """K = 20: the verification pass has 21 tokens per series, more than one 16-query tile, so its
    keys go to the cache through the append kernel and the attention runs in its multi-tile mode at
    ragged per-series positions, round after round (rows of rejected proposals are overwritten)."""
    wl = workload("C1", batch=4, horizon=96 * 6)
    for mode in (1, 0):
        run_and_compare(wl, 20, 2.0, 17, [0, 1, 2, 3], exec_mode=mode)


def test_many_series_short_rows_one_warp_per_series_and_head_bf16():
    """Enough (series, head) pairs on short rows for the attention mode that gives each warp a pair
    of its own, with a pair count that is not a multiple of the four warps of a CTA (199 x 6)."""
    wl = workload("C1", batch=199, horizon=96 * 3, target=Arch(2, 192, 6, 384), draft=Arch(1, 192, 6, 384),
                  draft_mode="layer_skip")
    run_and_compare(wl, 3, 1.0, 9, [0, 100, 198])


@pytest.mark.parametrize("B", [257, 340])
def test_many_series_long_rows_one_warp_per_series_and_head_bf16(B):
    """C4's row lengths with more than a thousand (series, head) pairs on small models: one warp per
    pair streams the whole row through its ring (257 x 4 and 340 x 4 pairs, four per CTA)."""
    wl = workload("C4", batch=B, horizon=32 * 5 + 3, target=Arch(2, 256, 4, 512), draft=Arch(1, 128, 2, 256))
    run_and_compare(wl, 4, 2.0, 5, [0, B // 2, B - 1])


@pytest.mark.parametrize("name,ids", [("C0", [0]), ("C1", [0, 7, 31]), ("C2", [3, 200])])
def test_draft_only_forecast_matches_oracle(name, ids):
    """Third arm of the matched three-way protocol: the draft model decoding on its own (Eq. 1)."""
    wl = workload(name)
    dec, tw, dw = make_decoder(wl)
    s, ctx = series_on_device(wl)
    out, st = dec.draft_only(ctx, wl.horizon)
    d = st.as_dict()
    assert d["device_status"] == 0 and d["rounds"] == wl.n_patches and d["patches_committed"] == wl.batch * wl.n_patches
    dec.close()
    tm, dm = parity.oracle_models(wl, tw, dw)
    want = orc.forecast_target_only(dm, s[list(ids)], wl.ctx_len, wl.horizon)
    kind, tol = parity.VALUE_TOL[wl.dtype]
    assert parity.per_series_errors(kind, out.cpu().numpy()[list(ids)], want).max() <= tol


@pytest.mark.parametrize("K,H,ctx_patches,B", [(32, 96 * 3, 2, 2), (1, 50, 2, 1), (5, 96, 3, 7), (8, 96 * 9 + 1, 7, 3)])
def test_edge_geometries_fp32(K, H, ctx_patches, B):
    """Degenerate and extreme geometries on the fp32 path: the largest block size the ABI allows (far
    more proposals than patches to commit), a horizon shorter than one patch, the shortest legal
    context (two patches), a single-patch horizon with K > T, a ragged last patch."""
    wl = workload("C0", batch=B, series_recipe="c1", horizon=H, ctx_len=96 * ctx_patches)
    for mode in (1, 0):
        res = run_and_compare(wl, K, 2.0, 11, range(B), exec_mode=mode)
        assert res["stats"]["rounds"] <= -(-H // 96)


@pytest.mark.parametrize("name,kw", [
    ("unequal_scales", dict(sigma_q=0.6)),
    ("sampled_proposals", dict(sample_proposals=1)),
    ("fallback_noise", dict(fallback_noise=0.3)),
    ("all_knobs", dict(sigma_q=0.8, fallback_noise=0.2, sample_proposals=1)),
    ("no_tempering", dict(no_tempering=1)),
])
@pytest.mark.parametrize("wl_name", ["C0", "C1"])
def test_general_rule_variants_match_oracle(wl_name, name, kw):
    """Sec. 3.3's sampled variants and Table 2's tempering ablation through the forecast call: sampled
    proposals (the draft continues from the sampled patch), fallback / bonus noise, sigma_q != sigma_p."""
    import paper_2511_18191_b200 as tsfm
    wl = workload("C0", batch=5, series_recipe="c1") if wl_name == "C0" else workload("C1", batch=6)
    K, tau, seed = wl.K, 1.5, 17
    dec, tw, dw = make_decoder(wl, batch=wl.batch)
    s, ctx = series_on_device(wl, wl.batch)
    v = tsfm.tsfm_variant(kw.get("sigma_q", 0.0), kw.get("fallback_noise", 0.0), kw.get("sample_proposals", 0),
                          kw.get("no_tempering", 0))
    base, _ = dec.forecast(ctx, wl.horizon, K, tau, seed)
    out, st = dec.forecast(ctx, wl.horizon, K, tau, seed, variant=v)
    d = check_stats(st, wl.batch, wl.n_patches, K)
    nacc, ell, logu = dec.last_trace(wl.batch, K)
    # replaying the default scheme afterwards on the same handle is unaffected by the variant call
    again, _ = dec.forecast(ctx, wl.horizon, K, tau, seed)
    np.testing.assert_array_equal(base.cpu().numpy(), again.cpu().numpy())
    dec.close()
    tm, dm = parity.oracle_models(wl, tw, dw)
    var = orc.Variant(sigma_q=kw.get("sigma_q") or None, sample_proposals=bool(kw.get("sample_proposals", 0)),
                      fallback_noise=kw.get("fallback_noise", 0.0), tempering=not kw.get("no_tempering", 0))
    res = parity.compare_forecast(wl, tm, dm, s, wl.horizon, K, tau, seed, out.cpu().numpy(), nacc, range(wl.batch),
                                  variant=var)
    if name != "unequal_scales":
        assert not np.allclose(out.cpu().numpy(), base.cpu().numpy())
    if name == "no_tempering":
        assert d["proposals_accepted"] == 0                     # acceptance collapses without the 1/d


def test_sampled_proposals_with_many_series_bf16():
    """Sampled proposals and fallback noise at 1024 series (C3 shape, small models): the draft head
    of such passes shares its weight loads between 8 series and adds the proposal noise itself."""
    import paper_2511_18191_b200 as tsfm
    wl = workload("C3", draft_eps=1e-2, horizon=96 * 4, target=Arch(2, 256, 4, 512), draft=Arch(2, 256, 4, 512))
    K, tau, seed, ids = 3, 1.5, 23, [0, 511, 1023]
    dec, tw, dw = make_decoder(wl, batch=wl.batch)
    s, ctx = series_on_device(wl, wl.batch)
    v = tsfm.tsfm_variant(0.8, 0.2, 1, 0)
    out, st = dec.forecast(ctx, wl.horizon, K, tau, seed, variant=v)
    check_stats(st, wl.batch, wl.n_patches, K)
    nacc, ell, logu = dec.last_trace(wl.batch, K)
    dec.close()
    tm, dm = parity.oracle_models(wl, tw, dw)
    var = orc.Variant(sigma_q=0.8, sample_proposals=True, fallback_noise=0.2, tempering=True)
    parity.compare_forecast(wl, tm, dm, s, wl.horizon, K, tau, seed, out.cpu().numpy(), nacc, ids, variant=var)


def test_tiny_tau_recovers_target_only_and_result_is_independent_of_batch_composition():
    wl = workload("C1")
    dec, tw, dw = make_decoder(wl)
    s, ctx = series_on_device(wl)
    ref, _ = dec.target_only(ctx, wl.horizon)
    out, st = dec.forecast(ctx, wl.horizon, wl.K, 1e-4, 5)
    d = st.as_dict()
    assert d["proposals_accepted"] == 0 and d["rounds"] == wl.n_patches
    assert parity.value_error("rel_rms", out.cpu().numpy(), ref.cpu().numpy().astype(np.float64)) < 1e-2
    # a series decoded alone (same series id 0) gives the same forecast as inside the batch
    full, _ = dec.forecast(ctx, wl.horizon, wl.K, 1.0, 5)
    solo, _ = dec.forecast(ctx[:1].contiguous(), wl.horizon, wl.K, 1.0, 5)
    assert parity.value_error("rel_rms", solo.cpu().numpy(), full[:1].cpu().numpy().astype(np.float64)) < 1e-2
    dec.close()


def test_argument_errors_are_reported_not_fatal():
    import paper_2511_18191_b200 as tsfm
    wl = workload("C0")
    dec, tw, dw = make_decoder(wl)
    s, ctx = series_on_device(wl)
    out = torch.empty((1, wl.horizon), device="cuda")
    for kw, code in [(dict(K=0), tsfm.TSFM_ERR_ARG), (dict(K=3), tsfm.TSFM_ERR_SHAPE),
                     (dict(tau=0.0), tsfm.TSFM_ERR_ARG), (dict(tau=float("nan")), tsfm.TSFM_ERR_ARG),
                     (dict(H=0), tsfm.TSFM_ERR_ARG), (dict(H=96 * 5), tsfm.TSFM_ERR_SHAPE),
                     (dict(ctx_len=100), tsfm.TSFM_ERR_SHAPE), (dict(ctx_len=96), tsfm.TSFM_ERR_SHAPE),
                     (dict(B=2), tsfm.TSFM_ERR_SHAPE)]:
        a = dict(B=1, ctx_len=wl.ctx_len, H=wl.horizon, K=2, tau=1.0)
        a.update(kw)
        with pytest.raises(tsfm.TsfmError) as e:
            tsfm.tsfm_spec_forecast(dec.h, ctx, a["B"], a["ctx_len"], a["H"], a["K"], a["tau"], 1, out, None)
        assert e.value.code == code, kw
    # the handle still works afterwards
    dec.forecast(ctx, wl.horizon, 2, 1.0, 1)
    dec.close()


def test_host_buffer_entry_points_match_device_ones():
    import paper_2511_18191_b200 as tsfm
    wl = workload("C0", batch=4, series_recipe="c1")      # fp32 path: bit-reproducible
    dec, tw, dw = make_decoder(wl)
    s, ctx = series_on_device(wl)
    out, _ = dec.forecast(ctx, wl.horizon, wl.K, 1.0, 3)
    h_in = torch.from_numpy(np.ascontiguousarray(s[:, :wl.ctx_len])).pin_memory()
    h_out = torch.empty((wl.batch, wl.horizon)).pin_memory()
    tsfm.tsfm_spec_forecast_host(dec.h, h_in, wl.batch, wl.ctx_len, wl.horizon, wl.K, 1.0, 3, h_out, None)
    np.testing.assert_array_equal(h_out.numpy(), out.cpu().numpy())
    ref, _ = dec.target_only(ctx, wl.horizon)
    tsfm.tsfm_target_only_forecast_host(dec.h, h_in, wl.batch, wl.ctx_len, wl.horizon, h_out, None)
    np.testing.assert_array_equal(h_out.numpy(), ref.cpu().numpy())
    dec.close()
