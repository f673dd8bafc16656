"""Parity at the full sizes of the workload, in the launch configuration the benchmark times.

The oracle cannot run 32 layers of the 7B shape in a test, so:
  * a 4-layer stack of the 7B WIDTHS (d=4096, 32x128 heads, ffn 11008, vocab 32000) at the full
    3376-token prompt, cuts entering layers 1/2/3 (3376/2364/1688/1013 rows), is compared with the
    oracle element by element, layer by layer (each layer against the oracle applied to the GPU's
    own input of that layer) and end to end (forced replay of the GPU's kept sets);
  * the full 32-layer model is checked on sampled outputs the oracle can compute one by one
    (whole layers 0, 7, 8 and 31 element by element, again on the GPU's own layer inputs, and the
    logits from its last hidden row) and on properties that hold at any size
    (scores sum to 1, selection bit-exact against the definition applied to the GPU's own scores,
    subset property, Aux = complement, counts);
  * prefill of a 4096-token prompt + 32 greedy decode steps, and the packed batch of 8 prompts of
    1024..4096 tokens, are checked through properties (each token computed at most once per layer,
    cache subset property, Aux = C_l minus C_{l+1}, packed batch == sequences run alone).
"""
import numpy as np
import pytest
import torch

import lazyllm_oracle as O
from paper_2407_14057_b200 import binding as B
from paper_2407_14057_b200 import build, synth
from helpers import rel_err, to_np, weights_to_np

pytestmark = pytest.mark.gpu
TOL = 2e-2
# End-to-end gates of the 32-layer run against the fp64 forced replay.  Measured: the residual stream's
# error grows like a random walk of one-layer roundings, 1.1e-2 after layer 0, 2.8e-2 after layer 7,
# 3.7e-2 after layer 15, 4.9e-2 after layer 23, 5.4e-2 after layer 31 (about 1.0e-2 x sqrt(layers)); logits
# 5.1e-2; Eq. 1 scores within 1.6e-3 absolute at every depth; the GPU's greedy token is the oracle's
# second-ranked token (logits of a random-init model are nearly flat) and the two top-10 sets coincide.
E2E_DRIFT_GATE = 0.08
E2E_LOGITS_GATE = 0.08
E2E_SCORE_ABS_GATE = 3e-3


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    B.lib()


@pytest.fixture(scope="module")
def model7b():
    W = synth.make_weights(synth.LLAMA7B, 2, bf16=True, device="cuda")
    yield W
    del W
    torch.cuda.empty_cache()


def _rows_entering(lengths, schedule, l):
    """Rows of every sequence that enter layer l (counts follow from lengths and schedule alone)."""
    rows = list(lengths)
    for e, bp in schedule:
        if e <= l:
            rows = [O.keep_count(n, bp, r) for n, r in zip(lengths, rows)]
    return rows


def _member_rows(packed, lengths, schedule, l_entering, seq):
    """Rows of sequence `seq` inside a packed [sum rows, d] tensor of the segment entering layer l_entering."""
    rows = _rows_entering(lengths, schedule, l_entering)
    a = sum(rows[:seq])
    assert packed.shape[0] == sum(rows)
    return packed[a:a + rows[seq]]


def _layer_inputs(eng, shape, emb, l, schedule, n, seq=0, lengths=None):
    """Rows and positions that ENTER layer l on the GPU (its own previous output)."""
    lengths = [n] if lengths is None else lengths
    pos = np.arange(n)
    for e, _ in schedule:
        if e <= l:
            pos = to_np(eng.lazy_get_kept(e, seq)).astype(np.int64)
    x = emb if l == 0 else to_np(_member_rows(eng.lazy_get_hidden(l - 1), lengths, schedule, l, seq))
    assert x.shape[0] == len(pos)
    return x, pos


def _check_layer_against_oracle(eng, shape, lw, emb, l, schedule, n, seq=0, lengths=None):
    """Layer l of the GPU run against the oracle applied to the GPU's own input of that layer: the
    per-layer form of the parity bound (2e-2 per tensor, scores 1e-3), free of the drift that a deep
    bf16 stack accumulates against an fp64 run.  seq / lengths pick one member of a packed batch."""
    lengths = [n] if lengths is None else lengths
    x_in, pos = _layer_inputs(eng, shape, emb, l, schedule, n, seq, lengths)
    keep = None
    for e, _ in schedule:
        if e == l + 1:
            keep = to_np(eng.lazy_get_kept(e, seq)).astype(np.int64)
    ref = O.layer_step(shape, lw, x_in, pos, keep_pos=keep)
    sc = to_np(eng.lazy_get_scores(l, seq))
    assert np.max(np.abs(sc - ref["scores"])) < 1e-3
    rel = np.abs(sc - ref["scores"]) / ref["scores"].clip(1e-30)
    assert np.max(rel) < 3e-2, (l, np.max(rel))       # same inputs on both sides: only one layer's rounding
    if keep is not None:                                # the cut: flips only at the threshold
        n_keep = len(keep)
        k_ref, _ = O.select_top(ref["scores"], n_keep, len(pos) - 1)
        diff = set(keep.tolist()) ^ set(pos[k_ref].tolist())
        tau = np.sort(ref["scores"][:-1])[::-1][n_keep - 2]
        s_of = dict(zip(pos.tolist(), ref["scores"].tolist()))
        for p in diff:
            assert abs(s_of[p] - tau) <= 3e-2 * tau and abs(s_of[p] - tau) <= 1e-3
        apos, ahid = eng.lazy_get_aux(l, seq)
        assert np.array_equal(to_np(apos), ref["aux_pos"])
        assert rel_err(to_np(ahid), ref["aux_rows"]) < TOL
    got = to_np(_member_rows(eng.lazy_get_hidden(l), lengths, schedule, l + 1, seq))
    assert rel_err(got, ref["hidden_out"]) < TOL, (l, rel_err(got, ref["hidden_out"]))
    kpos, kk, vv = eng.lazy_get_kv(l, seq)
    assert np.array_equal(to_np(kpos), pos)
    assert rel_err(to_np(kk), ref["k"].reshape(len(pos), -1)) < TOL
    assert rel_err(to_np(vv), ref["v"].reshape(len(pos), -1)) < TOL
    return ref


def test_7b_widths_four_layers_full_prompt_vs_oracle():
    shape = synth.LLAMA7B.with_layers(4)
    schedule = ((1, 7000), (2, 5000), (3, 3000))
    n = 3376
    W = synth.make_weights(shape, 3, bf16=True)
    Wn = weights_to_np(W)
    ids = synth.make_prompt(shape.vocab, n, 4)
    Wd = {k: v.cuda() for k, v in W.items() if k != "layers"}
    Wd["layers"] = [{k: v.cuda() for k, v in lw.items()} for lw in W["layers"]]
    eng = B.LazyPrefill(shape, Wd, schedule, torch.bfloat16, 1, n, debug_capture=True)
    logits = torch.empty((1, shape.vocab), dtype=torch.float32, device="cuda")
    eng.lazy_prefill_run(ids.cuda(), [0, n], logits)
    eng.lazy_sync_status()
    kept = {e: to_np(eng.lazy_get_kept(e, 0)).astype(np.int64) for e, _ in schedule}
    assert [len(kept[e]) for e, _ in schedule] == [2364, 1688, 1013]
    emb = Wn["tok_embed"][to_np(ids)]
    last = None
    for l in range(shape.n_layers):                     # every layer, element by element
        last = _check_layer_against_oracle(eng, shape, Wn["layers"][l], emb, l, schedule, n)
    ref_logits = O.lm_head(shape, Wn, to_np(eng.lazy_get_hidden(3))[-1])
    assert rel_err(to_np(logits[0]), ref_logits) < TOL
    # end to end against the oracle replayed on the GPU's kept sets: two layers deep the accumulated
    # bf16 drift is still inside the single-tensor bound; deeper it is reported, not gated
    replay = O.prefill(shape, Wn, to_np(ids), schedule, forced_keep=kept)
    drift = [rel_err(to_np(eng.lazy_get_hidden(l)), replay.hidden_out[l]) for l in range(4)]
    print("end-to-end drift per layer:", drift, "logits", rel_err(to_np(logits[0]), replay.logits))
    assert drift[0] < TOL and drift[1] < TOL
    assert all(d < 2 * TOL for d in drift) and rel_err(to_np(logits[0]), replay.logits) < 2 * TOL
    for l in range(4):
        assert np.max(np.abs(to_np(eng.lazy_get_scores(l, 0)) - replay.scores[l])) < 1e-3
    eng.close()


def _check_selection_properties(eng, n, schedule, seq, n_layers):
    prev = np.arange(n)
    for e, bp in schedule:
        kept = to_np(eng.lazy_get_kept(e, seq)).astype(np.int64)
        n_keep = O.keep_count(n, bp, len(prev))
        assert len(kept) == n_keep and kept[-1] == n - 1 and np.all(np.diff(kept) > 0)
        assert set(kept.tolist()) <= set(prev.tolist())
        sc = to_np(eng.lazy_get_scores(e - 1, seq))
        assert sc.shape == prev.shape and abs(float(sc.sum()) - 1.0) < 2e-3 and sc.min() >= 0
        k_def, d_def = O.select_top(sc, n_keep, len(prev) - 1)       # the definition on the GPU's own scores
        assert np.array_equal(kept, prev[k_def])
        apos, _ = eng.lazy_get_aux(e - 1, seq)
        assert np.array_equal(to_np(apos), prev[d_def])
        prev = kept
    return prev


def test_7b_full_depth_prefill_sampled_and_properties(model7b):
    shape, schedule, n = synth.LLAMA7B, synth.SCHEDULE_7B, 3376
    ids = synth.make_prompt(shape.vocab, n, 100)
    eng = B.LazyPrefill(shape, model7b, schedule, torch.bfloat16, 1, n, debug_capture=True)
    logits = torch.empty((1, shape.vocab), dtype=torch.float32, device="cuda")
    eng.lazy_prefill_run(ids.cuda(), [0, n], logits)
    eng.lazy_sync_status()
    _check_selection_properties(eng, n, schedule, 0, shape.n_layers)
    st = eng.lazy_get_stats()
    rows = [st.rows_computed[l] for l in range(32)]
    assert rows == [3376] * 8 + [2364] * 8 + [1688] * 8 + [1013] * 8
    assert torch.isfinite(logits).all()
    # sampled LAYERS of the full-depth run, each against the oracle on the GPU's own layer input:
    # the first layer, the layer that holds the first cut, the one after it, and the last one
    emb = to_np(model7b["tok_embed"][ids.long().cuda()])
    for l in (0, 7, 8, 31):
        lw = {k: to_np(v) for k, v in model7b["layers"][l].items()}
        _check_layer_against_oracle(eng, shape, lw, emb, l, schedule, n)
    ref_logits = O.lm_head(shape, {"g_final": to_np(model7b["g_final"]), "w_lm_head": to_np(model7b["w_lm_head"])},
                           to_np(eng.lazy_get_hidden(31))[-1])
    assert rel_err(to_np(logits[0]), ref_logits) < TOL
    # determinism: the same call three more times gives the same bits (no race between the warp
    # roles of the tensor-core kernels shows up as run-to-run noise)
    first = logits.clone()
    kept_first = [to_np(eng.lazy_get_kept(e, 0)) for e, _ in schedule]
    h_first = eng.lazy_get_hidden(31).clone()
    for _ in range(3):
        eng.lazy_prefill_run(ids.cuda(), [0, n], logits)
        eng.lazy_sync_status()
        assert torch.equal(logits, first)
        assert torch.equal(eng.lazy_get_hidden(31), h_first)
        for (e, _), k0 in zip(schedule, kept_first):
            assert np.array_equal(to_np(eng.lazy_get_kept(e, 0)), k0)
    eng.close()


def test_7b_full_depth_forced_replay_end_to_end_drift(model7b):
    """The whole 32-layer, 3376-token pruned prefill against the fp64 oracle replayed on the GPU's three
    kept sets (a chain of `layer_step` calls, one layer's weights widened at a time: the same arithmetic as
    `prefill` with forced sets).  Records the drift of the residual stream per layer, the error of the
    first-token logits and whether the greedy token agrees.  The per-tensor 2e-2 bound is a one-layer
    bound (see _check_layer_against_oracle); end to end the bf16 rounding of 32 layers accumulates, and the
    gates below are what the measurement supports, with margin."""
    shape, schedule, n = synth.LLAMA7B, synth.SCHEDULE_7B, 3376
    ids = synth.make_prompt(shape.vocab, n, 100)
    eng = B.LazyPrefill(shape, model7b, schedule, torch.bfloat16, 1, n, debug_capture=True)
    logits = torch.empty((1, shape.vocab), dtype=torch.float32, device="cuda")
    eng.lazy_prefill_run(ids.cuda(), [0, n], logits)
    eng.lazy_sync_status()
    kept = {e: to_np(eng.lazy_get_kept(e, 0)).astype(np.int64) for e, _ in schedule}
    x = to_np(model7b["tok_embed"][ids.long().cuda()]).astype(np.float64)
    pos = np.arange(n)
    drift, score_abs, score_rel = [], [], []
    for l in range(shape.n_layers):
        lw = {k: to_np(v) for k, v in model7b["layers"][l].items()}
        ref = O.layer_step(shape, lw, x, pos, keep_pos=kept.get(l + 1))
        drift.append(rel_err(to_np(eng.lazy_get_hidden(l)), ref["hidden_out"]))
        sc = to_np(eng.lazy_get_scores(l, 0))
        score_abs.append(float(np.max(np.abs(sc - ref["scores"]))))
        score_rel.append(float(np.max(np.abs(sc - ref["scores"]) / ref["scores"].clip(1e-30))))
        x, pos = ref["hidden_out"], ref["pos_out"]
    ref_logits = O.lm_head(shape, {"g_final": to_np(model7b["g_final"]), "w_lm_head": to_np(model7b["w_lm_head"])},
                           x[-1])
    got = to_np(logits[0]).astype(np.float64)
    lerr = rel_err(got, ref_logits)
    order = np.argsort(-ref_logits)
    rank_of_gpu_argmax = int(np.nonzero(order == int(np.argmax(got)))[0][0])
    top10 = len(set(order[:10].tolist()) & set(np.argsort(-got)[:10].tolist()))
    print("e2e drift per layer:", " ".join(f"{d:.4f}" for d in drift))
    print(f"e2e logits rel err {lerr:.4f}; greedy token equal: {rank_of_gpu_argmax == 0} "
          f"(GPU argmax is the oracle's rank {rank_of_gpu_argmax}); top-10 overlap {top10}/10; "
          f"scores: max abs {max(score_abs):.2e}, max rel {max(score_rel):.3f}")
    assert drift[0] < TOL and drift[1] < TOL                   # no accumulation yet: the one-layer bound
    print("e2e score abs err per layer:", " ".join(f"{a:.1e}" for a in score_abs))
    assert max(score_abs[:8]) < 1e-3                           # Eq. 1 scores before the first cut: the one-layer bound
    assert max(score_abs) < E2E_SCORE_ABS_GATE                 # deeper: inputs have drifted, see the gates above
    assert all(d < 1.6e-2 * (l + 1) ** 0.5 + 4e-3 for l, d in enumerate(drift))   # random-walk growth, not linear
    assert max(drift) < E2E_DRIFT_GATE and lerr < E2E_LOGITS_GATE
    assert rank_of_gpu_argmax < 3 and top10 >= 8
    eng.close()


def test_7b_prefill_4096_then_32_decode_steps_properties(model7b):
    shape, schedule, n, steps = synth.LLAMA7B, synth.SCHEDULE_7B, 4096, 32
    ids = synth.make_prompt(shape.vocab, n, 101)
    eng = B.LazyPrefill(shape, model7b, schedule, torch.bfloat16, 1, n, max_new_tokens=steps)
    logits = torch.empty((1, shape.vocab), dtype=torch.float32, device="cuda")
    nxt = torch.empty(1, dtype=torch.int32, device="cuda")
    eng.lazy_prefill_run(ids.cuda(), [0, n], logits)
    eng.lazy_sync_status()
    kept = _check_selection_properties(eng, n, schedule, 0, shape.n_layers)
    assert [len(to_np(eng.lazy_get_kept(e, 0))) for e, _ in schedule] == [2868, 2048, 1229]
    tok = torch.argmax(logits, dim=1).to(torch.int32)
    baseline_kv = None
    total_revived = 0
    for step in range(steps):
        eng.lazy_decode_step(tok, logits, nxt)
        eng.lazy_sync_status()
        p = n + step
        assert torch.isfinite(logits).all()
        assert int(nxt[0]) == int(torch.argmax(logits[0]))
        tok = nxt.clone()
        st = eng.lazy_get_stats()
        kv = [st.kv_rows[l] for l in range(32)]
        assert kv[0] == p + 1 and all(kv[l + 1] <= kv[l] for l in range(31))   # usage bounded by the baseline
        if baseline_kv is not None:
            assert all(a >= b for a, b in zip(kv, baseline_kv))                   # caches only grow
        baseline_kv = kv
        for e, bp in schedule:
            sel = to_np(eng.lazy_get_kept(e, 0))
            assert len(sel) == O.keep_count(p + 1, bp, p + 1) and sel[-1] == p and np.all(np.diff(sel) > 0)
            total_revived += st.revived[e]
            assert st.aux_rows[e - 1] == kv[e - 1] - kv[e]                        # Aux = C_l minus C_{l+1}
        if step in (0, 15, 31):
            prev = None
            for l in (0, 7, 8, 15, 16, 23, 24, 31):
                cnt_pos = to_np(eng.lazy_get_kv(l, 0)[0])
                assert len(set(cnt_pos.tolist())) == len(cnt_pos) == kv[l]        # at most once per layer
                if prev is not None:
                    assert set(cnt_pos.tolist()) <= prev
                prev = set(cnt_pos.tolist())
            sc = to_np(eng.lazy_get_scores(7, 0))
            k_def, _ = O.select_top(sc, len(to_np(eng.lazy_get_kept(8, 0))), len(sc) - 1)
            assert np.array_equal(to_np(eng.lazy_get_kept(8, 0)), k_def)          # context of layers 0..7 is 0..p
    assert total_revived > 0
    eng.close()


def test_7b_varlen_batch_of_8_vs_oracle_and_vs_sequences_run_alone(model7b):
    shape, schedule = synth.LLAMA7B, synth.SCHEDULE_7B
    lengths = synth.make_varlen_lengths(8, 1024, 4096, seed=4)
    ids, cu = synth.make_varlen_batch(shape.vocab, lengths, seed=5)
    eng = B.LazyPrefill(shape, model7b, schedule, torch.bfloat16, 8, sum(lengths), debug_capture=True)
    logits = torch.empty((8, shape.vocab), dtype=torch.float32, device="cuda")
    d_ids = ids.cuda()
    eng.lazy_prefill_run(d_ids, cu, logits)
    eng.lazy_sync_status()
    assert torch.isfinite(logits).all()
    kept_batch = []
    for s in range(8):
        _check_selection_properties(eng, lengths[s], schedule, s, shape.n_layers)
        kept_batch.append([to_np(eng.lazy_get_kept(e, s)) for e, _ in schedule])
    # one member of the packed batch against the ORACLE, element by element, on the GPU's own layer inputs:
    # the first layer, the layer that holds the first cut and the one after it (a member in the middle of
    # the packing, so that its rows start inside a GEMM tile and an attention launch of their own)
    m = 3
    emb = to_np(model7b["tok_embed"][d_ids[cu[m]:cu[m + 1]].long()])
    for l in (0, 7, 8):
        lw = {k: to_np(v) for k, v in model7b["layers"][l].items()}
        _check_layer_against_oracle(eng, shape, lw, emb, l, schedule, lengths[m], seq=m, lengths=lengths)
    h_last = to_np(_member_rows(eng.lazy_get_hidden(31), lengths, schedule, 32, m))[-1]
    ref_logits = O.lm_head(shape, {"g_final": to_np(model7b["g_final"]), "w_lm_head": to_np(model7b["w_lm_head"])},
                           h_last)
    assert rel_err(to_np(logits[m]), ref_logits) < TOL
    score_batch = {s: [to_np(eng.lazy_get_scores(e - 1, s)) for e, _ in schedule] for s in (0, 3, 7)}
    eng.close()
    del eng
    torch.cuda.empty_cache()
    # Sequences are independent, so a member run alone must reproduce the batch.  Not bit for bit: which
    # output tiles of a GEMM get their K loop split across SMs depends on the total row count, and a split
    # tile adds its fp32 partial sums in another order.  The comparison is therefore made cut by cut on the same
    # token sets: the solo run is handed the batch's kept sets for the earlier cuts and selects freely at cut i.
    # The bf16 roundings of every layer fall differently in the two runs, so the two score vectors agree to a
    # few per cent, less well the deeper the cut (measured: differing tokens lie within 1.5 % / 3.1 % / 8.0 % of
    # the threshold at the cuts entering layers 8 / 16 / 24, and 0.3 % / 0.8 % / 1.7 % of the kept tokens differ).
    # The two sets may therefore differ only in tokens whose score lies within 4 % / 8 % / 16 % of the
    # threshold, and in at most 4 % of the tokens.  With all three sets handed over, the logits are those of two
    # bf16 runs of 32 layers whose roundings differ in places: each lies about 5e-2 from exact arithmetic (see
    # E2E_LOGITS_GATE), they lie 3.0e-2 from each other (measured), and are held to twice the one-tensor bound.
    solo = B.LazyPrefill(shape, model7b, schedule, torch.bfloat16, 1, max(lengths))
    lg = torch.empty((1, shape.vocab), dtype=torch.float32, device="cuda")
    for s in (0, 3, 7):
        p_ids = d_ids[cu[s]:cu[s + 1]].contiguous()
        for i, (e, _) in enumerate(schedule):
            for j in range(i):
                solo.lazy_set_forced_keep(schedule[j][0], 0, torch.tensor(kept_batch[s][j], dtype=torch.int32).cuda())
            solo.lazy_prefill_run(p_ids, [0, lengths[s]], lg)
            solo.lazy_sync_status()
            a, b = to_np(solo.lazy_get_kept(e, 0)), kept_batch[s][i]
            assert len(a) == len(b)
            cand = np.arange(lengths[s]) if i == 0 else kept_batch[s][i - 1]
            sc = score_batch[s][i]
            assert sc.shape == cand.shape
            tau = np.sort(sc[:-1])[::-1][len(b) - 2]
            s_of = dict(zip(cand.tolist(), sc.tolist()))
            diff = set(a.tolist()) ^ set(b.tolist())
            worst = max([abs(s_of[p] - tau) / tau for p in diff], default=0.0)
            print(f"seq {s} cut entering layer {e}: {len(diff) // 2} of {len(b)} tokens differ, all within "
                  f"{100 * worst:.2f} % of the threshold")
            assert worst <= (4e-2, 8e-2, 16e-2)[i] and len(diff) // 2 <= 0.04 * len(b), (s, e, worst, len(diff))
        for j, (e, _) in enumerate(schedule):
            solo.lazy_set_forced_keep(e, 0, torch.tensor(kept_batch[s][j], dtype=torch.int32).cuda())
        solo.lazy_prefill_run(p_ids, [0, lengths[s]], lg)
        solo.lazy_sync_status()
        both = rel_err(to_np(lg[0]), to_np(logits[s]).astype(np.float64))
        print(f"seq {s} logits, batch member vs run alone on the same kept sets: {both:.4f}")
        assert both < 2 * TOL
        # free-running, for the record: rounding noise moves ranks next to the threshold, and a different
        # set at one cut changes every later score a little
        solo.lazy_prefill_run(p_ids, [0, lengths[s]], lg)
        solo.lazy_sync_status()
        ov = [len(np.intersect1d(to_np(solo.lazy_get_kept(e, 0)), kept_batch[s][i])) / len(kept_batch[s][i])
              for i, (e, _) in enumerate(schedule)]
        print(f"seq {s} free-running kept-set overlap with the batch run per cut: {[round(o, 4) for o in ov]}")
        assert ov[0] >= 0.99 and min(ov) >= 0.90
    solo.close()
