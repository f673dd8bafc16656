"""End-to-end parity of the token-pruned prefill (and the single-layer pruning op) against the
CPU oracle, through the C ABI.

Protocol.  The GPU run selects its own kept sets.  (1) Scores are compared directly wherever both
sides still hold the same rows; (2) a kept-set difference is accepted only for tokens whose oracle
score lies within the band of the threshold (1e-3 absolute as the stated bound, and a relative
band that is not vacuous at long prompts); (3) because one flipped token changes every deeper
tensor, hidden states, caches and logits are compared with the oracle re-run on the GPU's kept
sets (forced replay); (4) the GPU is also re-run on the oracle's kept sets.
Tolerances: per-tensor max|a-b| <= tol*max|b| with tol 2e-2 (bf16) / 1e-4 (fp32); scores 1e-3.
"""
import numpy as np
import pytest
import torch

import lazyllm_oracle as O
from paper_2407_14057_b200 import binding as B
from paper_2407_14057_b200 import build, synth
from helpers import rel_err, to_np, weights_to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    B.lib()


def _to_cuda(W):
    out = {k: v.cuda() for k, v in W.items() if k != "layers"}
    out["layers"] = [{k: v.cuda() for k, v in lw.items()} for lw in W["layers"]]
    return out


# With e4m3 projections the two sides quantise activations that differ by bf16 rounding noise (attention outputs,
# SwiGLU outputs: about half a per cent), and an element that falls on the other side of a rounding boundary moves
# by a whole e4m3 step (6 to 12 % of its value).  The disagreement feeds the next projection's quantiser, so
# within one layer it grows to the level of the e4m3 noise itself and then stays there: measured 3.5-5.5 % of the
# tensor in the root-mean-square sense and 3-7 % of its maximum element by element at 512 features, 9 % at the
# 4096 / 11008-feature widths, at every depth (it does not accumulate).  Two runs in this mode cannot agree
# more closely than that; what pins the arithmetic exactly are the step-level tests (bit-exact quantiser,
# product of given codes to 1e-2).  Here tensors are held to 2e-1 of their maximum and 1.5e-1 root-mean-square,
# scores to 3e-3, kept-set differences to a 15 % band.
FP8_TOL, FP8_BAND, FP8_RMS, FP8_SCORE_ABS = 2e-1, 1.5e-1, 1.5e-1, 3e-3


def _tols(dtype, fp8=False):
    if fp8:
        return FP8_TOL, FP8_BAND
    return (1e-4, 1e-5) if dtype == torch.float32 else (2e-2, 3e-2)   # tensor tol, relative score band


def _check_set_difference(gpu_pos, ref_pos, ref_scores, ref_score_pos, band_rel, band_abs=1e-3):
    """Tokens kept by one side only must sit at the threshold."""
    g, r = set(gpu_pos.tolist()), set(ref_pos.tolist())
    assert len(g) == len(r)
    diff = g ^ r
    if not diff:
        return 0
    s_of = dict(zip(ref_score_pos.tolist(), ref_scores.tolist()))
    last = int(ref_score_pos[-1])
    tau = min(s_of[p] for p in r if p != last)
    for p in diff:
        assert abs(s_of[p] - tau) <= band_abs, (p, s_of[p], tau)
        assert abs(s_of[p] - tau) <= band_rel * tau, (p, s_of[p], tau)
    return len(diff)


def run_model_case(shape, schedule, lengths, dtype, seed, perturb=True, max_new=0):
    bf16 = dtype == torch.bfloat16
    fp8 = getattr(shape, "fp8", False)
    tol, band = _tols(dtype, fp8)
    score_abs = FP8_SCORE_ABS if fp8 else 1e-3
    W = synth.make_weights(shape, seed, bf16=bf16)
    if perturb:
        synth.perturb_gains(W, seed + 100)
    q8 = synth.quantize_projections_e4m3(W) if fp8 else None     # W now holds the de-quantised weights
    Wn = weights_to_np(W)
    ids, cu = synth.make_varlen_batch(shape.vocab, lengths, seed + 1)
    n_seqs = len(lengths)
    eng = B.LazyPrefill(shape, _to_cuda(W), schedule, dtype, max_seqs=n_seqs,
                        max_prompt_tokens=sum(lengths), max_new_tokens=max_new, debug_capture=True)
    if fp8:
        eng.lazy_set_fp8_weights({"layers": [{k: (c.cuda(), s) for k, (c, s) in lq.items()} for lq in q8["layers"]]})
    logits = torch.empty((n_seqs, shape.vocab), dtype=torch.float32, device="cuda")
    d_ids = ids.cuda()
    eng.lazy_prefill_run(d_ids, cu, logits)
    eng.lazy_sync_status()
    stats = eng.lazy_get_stats()
    points = [e for e, _ in schedule]
    flips = 0
    hidden = [to_np(eng.lazy_get_hidden(l)) for l in range(shape.n_layers)]
    row_off = [0] * shape.n_layers
    for s in range(n_seqs):
        sid = to_np(ids)[cu[s]:cu[s + 1]]
        free = O.prefill(shape, Wn, sid, schedule)
        gpu_kept = {e: to_np(eng.lazy_get_kept(e, s)).astype(np.int64) for e in points}
        # (1) scores before the first cut see identical rows on both sides
        first = points[0] if points else shape.n_layers
        for l in range(first):
            sc = to_np(eng.lazy_get_scores(l, s))
            assert np.max(np.abs(sc - free.scores[l])) < score_abs
            assert abs(sc.sum() - 1.0) < 1e-3 and sc.min() >= 0
        # (2)+(3) walk the cuts: compare against the oracle replayed on the GPU's sets so far
        replay = O.prefill(shape, Wn, sid, schedule, forced_keep=gpu_kept)
        prev = None
        for e in points:
            partial = {k: v for k, v in gpu_kept.items() if k < e}
            ref = O.prefill(shape, Wn, sid, schedule, forced_keep=partial) if partial else free
            flips += _check_set_difference(gpu_kept[e], ref.kept_pos[e], ref.scores[e - 1],
                                           ref.score_pos[e - 1], band, score_abs)
            assert np.all(np.diff(gpu_kept[e]) > 0) and gpu_kept[e][-1] == len(sid) - 1
            if prev is not None:
                assert set(gpu_kept[e].tolist()) <= set(prev.tolist())       # subset property
            prev = gpu_kept[e]
        for l in range(shape.n_layers):
            sc = to_np(eng.lazy_get_scores(l, s))
            assert sc.shape == replay.scores[l].shape
            assert np.max(np.abs(sc - replay.scores[l])) < score_abs
            n_l = replay.hidden_out[l].shape[0]
            got = hidden[l][row_off[l]:row_off[l] + n_l]
            row_off[l] += n_l
            assert rel_err(got, replay.hidden_out[l]) < tol, (l, rel_err(got, replay.hidden_out[l]))
            if fp8:
                rms = float(np.sqrt(np.mean((got - replay.hidden_out[l]) ** 2) / np.mean(replay.hidden_out[l] ** 2)))
                assert rms < FP8_RMS, (l, rms)
            kpos, kk, vv = eng.lazy_get_kv(l, s)
            assert np.array_equal(to_np(kpos), replay.rows_pos[l])
            kr, vr = replay.layers[l].rows(replay.rows_pos[l])
            assert rel_err(to_np(kk), kr.reshape(len(kpos), -1)) < tol
            assert rel_err(to_np(vv), vr.reshape(len(kpos), -1)) < tol
            apos, ahid = eng.lazy_get_aux(l, s)
            want = sorted(replay.layers[l].aux.keys())
            assert to_np(apos).tolist() == want
            if want:
                ref_rows = np.stack([replay.layers[l].aux[p] for p in want])
                assert rel_err(to_np(ahid), ref_rows) < tol
                rev = eng.aux_cache_revive(l, s, apos[: min(5, len(want))].contiguous())
                assert torch.equal(rev, ahid[: min(5, len(want))])
        assert rel_err(to_np(logits[s]), replay.logits) < tol
        # (4) GPU on the oracle's own kept sets
        for e in points:
            eng.lazy_set_forced_keep(e, s, torch.tensor(free.kept_pos[e], dtype=torch.int32).cuda())
    if points:
        logits2 = torch.empty_like(logits)
        eng.lazy_prefill_run(d_ids, cu, logits2)
        eng.lazy_sync_status()
        for s in range(n_seqs):
            free = O.prefill(shape, Wn, to_np(ids)[cu[s]:cu[s + 1]], schedule)
            for e in points:
                assert np.array_equal(to_np(eng.lazy_get_kept(e, s)), free.kept_pos[e])
            assert rel_err(to_np(logits2[s]), free.logits) < tol
            assert int(torch.argmax(logits2[s])) == O.greedy(free.logits) or bf16
    assert stats.kernel_launches > 0
    eng.close()
    return flips


def test_tiny_fp32_config():
    """2 layers, d=256, 4x64 heads, ffn 688, vocab 1024, one 256-token prompt, keep 50 % entering
    layer 1, next-token logits; fp32 mode."""
    flips = run_model_case(synth.TINY, synth.SCHEDULE_TINY, [256], torch.float32, seed=0, perturb=False)
    assert flips == 0


def test_tiny_fp32_three_cuts_and_ragged_lengths():
    shape = synth.TINY.with_layers(4)
    run_model_case(shape, ((1, 7000), (2, 5000), (3, 3000)), [129], torch.float32, seed=3)


def test_fp32_varlen_batch():
    shape = synth.TINY.with_layers(3)
    run_model_case(shape, ((1, 6000), (2, 2500)), [70, 1, 33, 150], torch.float32, seed=4)


def test_full_keep_schedule_is_standard_prefill():
    shape = synth.TINY
    W = synth.make_weights(shape, 7, bf16=False)
    ids = synth.make_prompt(shape.vocab, 100, 8)
    out = []
    for sched in ((), ((1, 10000),)):
        eng = B.LazyPrefill(shape, _to_cuda(W), sched, torch.float32, 1, 100)
        lg = torch.empty((1, shape.vocab), dtype=torch.float32, device="cuda")
        eng.lazy_prefill_run(ids.cuda(), [0, 100], lg)
        eng.lazy_sync_status()
        out.append(lg.cpu())
        eng.close()
    assert torch.equal(out[0], out[1])
    ref = O.prefill(shape, weights_to_np(W), to_np(ids), ())
    assert rel_err(to_np(out[0][0]), ref.logits) < 1e-4


def test_small_bf16_model_multi_tile():
    """head_dim 128 model on the tensor-core kernels: 300 rows = several GEMM and attention tiles
    with ragged tails, three cuts."""
    run_model_case(synth.SMALL, ((1, 7000), (2, 5000), (3, 3000)), [300], torch.bfloat16, seed=5)


def test_small_bf16_varlen_batch():
    run_model_case(synth.SMALL.with_layers(3), ((1, 6000), (2, 3000)), [200, 65, 1, 131], torch.bfloat16, seed=6)


def test_capacity_and_argument_errors():
    shape = synth.TINY
    W = _to_cuda(synth.make_weights(shape, 1, bf16=False))
    eng = B.LazyPrefill(shape, W, synth.SCHEDULE_TINY, torch.float32, 1, 64)
    lg = torch.empty((1, shape.vocab), dtype=torch.float32, device="cuda")
    ids = synth.make_prompt(shape.vocab, 65, 1).cuda()
    with pytest.raises(B.LazyError) as e:
        eng.lazy_prefill_run(ids, [0, 65], lg)
    assert e.value.status == -3
    with pytest.raises(B.LazyError) as e:
        eng.lazy_prefill_run(ids, [0, 10, 20], lg)                    # two sequences, room for one
    assert e.value.status == -3
    with pytest.raises(B.LazyError) as e:
        eng.lazy_get_kept(1, 0)                                       # nothing has run yet
    assert e.value.status == -7
    bad = ids.clone()
    bad[3] = shape.vocab + 5                                          # id out of range: reported
    eng.lazy_prefill_run(bad[:64].contiguous(), [0, 64], lg)
    with pytest.raises(B.LazyError) as e:
        eng.lazy_sync_status()
    assert e.value.status == -1
    eng.lazy_prefill_run(ids[:64].contiguous(), [0, 64], lg)
    eng.lazy_sync_status()
    pos, _ = eng.lazy_get_aux(0, 0)
    kept = eng.lazy_get_kept(1, 0)
    with pytest.raises(B.LazyError) as e:
        eng.aux_cache_revive(0, 0, kept[:1].contiguous())             # a kept token is not in Aux
    assert e.value.status == -4
    assert eng.aux_cache_revive(0, 0, pos[:3].contiguous()).shape == (3, shape.d_model)
    eng.close()


# ------------------------------------------------------------------------------------------ prune op
def _prune_case(dtype, n, H, dh, keep_bp, seed, pos=None):
    d = H * dh
    bf16 = dtype == torch.bfloat16
    tol, band = _tols(dtype)
    shape = synth.ModelShape(1, d, H, dh, 8, 8)
    g = torch.Generator().manual_seed(seed)
    lw = {"w_qkv": torch.empty(3 * d, d).normal_(0, 0.02, generator=g).to(dtype),
          "w_o": torch.empty(d, d).normal_(0, 0.02, generator=g).to(dtype),
          "g_attn": torch.ones(d, dtype=dtype)}
    x = synth.make_hidden(n, d, seed + 1, bf16)
    pos = torch.arange(n, dtype=torch.int32) if pos is None else pos
    max_pos = int(pos.max()) + 1
    out = B.lazy_prune_op(x.cuda(), pos.cuda(), lw["w_qkv"].cuda(), lw["w_o"].cuda(), lw["g_attn"].cuda(),
                          H, dh, keep_bp, max_pos)
    B.lazy_device_status()
    lwn = {k: to_np(v) for k, v in lw.items()}
    ref = O.prune_op(shape, lwn, to_np(x), to_np(pos), keep_bp)
    sc = to_np(out["scores"])
    assert np.max(np.abs(sc - ref["scores"])) < 1e-3
    assert np.max(np.abs(sc - ref["scores"]) / ref["scores"].clip(1e-30)) < band
    keep = to_np(out["keep_idx"]).astype(np.int64)
    drop = to_np(out["drop_idx"]).astype(np.int64)[: out["n_drop"]]
    assert len(keep) == len(ref["keep"]) and keep[-1] == n - 1
    assert sorted(keep.tolist() + drop.tolist()) == list(range(n))
    flips = _check_set_difference(keep, ref["keep"], ref["scores"], np.arange(n), band)
    # the selection itself is bit-exact given the GPU's own scores
    k2, d2 = O.select_top(sc, len(keep), n - 1)
    assert np.array_equal(keep, k2) and np.array_equal(drop, d2)
    rep = O.prune_op(shape, lwn, to_np(x), to_np(pos), keep_bp, forced_keep_rows=keep)
    assert rel_err(to_np(out["hidden_kept"]), rep["hidden_kept"]) < tol
    assert rel_err(to_np(out["k_kept"]), rep["k_kept"].reshape(len(keep), d)) < tol
    assert rel_err(to_np(out["v_kept"]), rep["v_kept"].reshape(len(keep), d)) < tol
    assert np.array_equal(to_np(out["pos_kept"]), rep["pos_kept"])
    if out["n_drop"]:
        assert rel_err(to_np(out["aux_hidden"])[: out["n_drop"]], rep["aux_rows"]) < tol
        assert np.array_equal(to_np(out["aux_pos"])[: out["n_drop"]], rep["aux_pos"])
    # GPU forced onto the oracle's set: gathered rows are exact copies of rows the op itself made
    forced = B.lazy_prune_op(x.cuda(), pos.cuda(), lw["w_qkv"].cuda(), lw["w_o"].cuda(), lw["g_attn"].cuda(),
                             H, dh, keep_bp, max_pos,
                             forced_keep_idx=torch.tensor(ref["keep"], dtype=torch.int32).cuda())
    B.lazy_device_status()
    assert np.array_equal(to_np(forced["keep_idx"]), ref["keep"])
    assert rel_err(to_np(forced["hidden_kept"]), ref["hidden_kept"]) < tol
    return flips


def test_prune_op_fp32_small():
    assert _prune_case(torch.float32, 200, 4, 64, 6000, seed=1) == 0


def test_prune_op_bf16_multi_tile_with_position_gaps():
    pos = torch.tensor(sorted(np.random.default_rng(3).choice(5000, 700, replace=False)), dtype=torch.int32)
    _prune_case(torch.bfloat16, 700, 4, 128, 6000, seed=2, pos=pos)


def test_prune_op_keep_everything_and_keep_one():
    _prune_case(torch.float32, 64, 4, 64, 10000, seed=4)
    _prune_case(torch.float32, 64, 4, 64, 1, seed=5)


def test_prune_op_full_size_bf16():
    """The single-layer pruning op at its full size: hidden [4096, 4096], 32 heads x 128, keep 60 %
    (2458 kept / 1638 to the Aux Cache)."""
    _prune_case(torch.bfloat16, 4096, 32, 128, 6000, seed=1)


# ----------------------------------------------------------------------------- threshold reading end to end
def _zero_query(W, layer, d):
    """q = 0 in one layer: every attention row is uniform, every Eq. 1 score equals 1/n exactly."""
    W["layers"][layer]["w_qkv"][:d] = 0


def test_threshold_selection_prefill_and_decode_with_ties_fp32():
    """The selection read as a threshold (pruned iff the score is smaller than the score at the scheduled rank):
    ties at the threshold all survive, so row counts depend on the data and the library reads them back at
    every point.  Layer 0 has a zero query projection, so all its scores tie: sequence by sequence the first
    cut prunes NOTHING under this reading (the count reading would keep 60 %), the later cuts have no ties and
    keep the scheduled counts.  Kept sets, hidden states, caches, Aux contents, logits and two decode steps
    against the oracle run with the same reading."""
    shape, schedule, lengths = synth.TINY.with_layers(3), ((1, 6000), (2, 3000)), [50, 9, 31]
    W = synth.make_weights(shape, 21, bf16=False)
    synth.perturb_gains(W, 121)
    _zero_query(W, 0, shape.d_model)
    Wn = weights_to_np(W)
    ids, cu = synth.make_varlen_batch(shape.vocab, lengths, 22)
    S = len(lengths)
    eng = B.LazyPrefill(shape, _to_cuda(W), schedule, torch.float32, S, sum(lengths), max_new_tokens=2,
                        debug_capture=True)
    eng.lazy_set_selection(True)
    logits = torch.empty((S, shape.vocab), dtype=torch.float32, device="cuda")
    nxt = torch.empty(S, dtype=torch.int32, device="cuda")
    eng.lazy_prefill_run(ids.cuda(), cu, logits)
    eng.lazy_sync_status()
    states = [O.prefill(shape, Wn, to_np(ids)[cu[s]:cu[s + 1]], schedule, selection="threshold") for s in range(S)]
    st = eng.lazy_get_stats()
    assert st.rows_computed[0] == sum(lengths) and st.rows_computed[1] == sum(lengths)     # nothing pruned at cut 1
    assert st.rows_computed[2] == sum(O.keep_count(n, 3000, n) for n in lengths)
    off = [0] * shape.n_layers
    for s in range(S):
        ref = states[s]
        assert len(ref.kept_pos[1]) == lengths[s]                                          # the oracle agrees
        for e, _ in schedule:
            assert np.array_equal(to_np(eng.lazy_get_kept(e, s)), ref.kept_pos[e])
        for l in range(shape.n_layers):
            assert np.max(np.abs(to_np(eng.lazy_get_scores(l, s)) - ref.scores[l])) < 1e-5
            n_l = ref.hidden_out[l].shape[0]
            got = to_np(eng.lazy_get_hidden(l))[off[l]:off[l] + n_l]
            off[l] += n_l
            assert rel_err(got, ref.hidden_out[l]) < 1e-4
            apos, _ = eng.lazy_get_aux(l, s)
            assert to_np(apos).tolist() == sorted(ref.layers[l].aux.keys())
        assert rel_err(to_np(logits[s]), ref.logits) < 1e-4
    tok = [O.greedy(s_.logits) for s_ in states]
    for step in range(2):
        ref_logits = [O.decode_step(shape, Wn, states[s], tok[s]) for s in range(S)]
        eng.lazy_decode_step(torch.tensor(tok, dtype=torch.int32).cuda(), logits, nxt)
        eng.lazy_sync_status()
        for s in range(S):
            assert rel_err(to_np(logits[s]), ref_logits[s]) < 1e-4, (step, s)
            for e, _ in schedule:
                assert np.array_equal(to_np(eng.lazy_get_kept(e, s)), states[s].kept_pos[e]), (step, s, e)
                assert sorted(to_np(eng.lazy_get_revived(e, s)).tolist()) == sorted(states[s].revived_pos[e].tolist())
            assert int(nxt[s]) == O.greedy(ref_logits[s])
        tok = [O.greedy(l) for l in ref_logits]
    # the count reading on the same inputs prunes at the first cut
    eng.lazy_set_selection(False)
    eng.lazy_prefill_run(ids.cuda(), cu, logits)
    eng.lazy_sync_status()
    assert eng.lazy_get_stats().rows_computed[1] == sum(O.keep_count(n, 6000, n) for n in lengths)
    eng.close()


def test_threshold_selection_equals_count_selection_without_ties_bf16():
    """Generic inputs have no ties at the threshold: both readings select the same sets and give the same bits."""
    shape, schedule, n = synth.SMALL, ((1, 7000), (2, 5000), (3, 3000)), 333
    W = _to_cuda(synth.make_weights(shape, 23, bf16=True))
    ids = synth.make_prompt(shape.vocab, n, 24).cuda()
    out = []
    for thr in (False, True):
        eng = B.LazyPrefill(shape, W, schedule, torch.bfloat16, 1, n)
        eng.lazy_set_selection(thr)
        lg = torch.empty((1, shape.vocab), dtype=torch.float32, device="cuda")
        eng.lazy_prefill_run(ids, [0, n], lg)
        eng.lazy_sync_status()
        out.append((lg.clone(), [to_np(eng.lazy_get_kept(e, 0)) for e, _ in schedule]))
        eng.close()
    assert all(np.array_equal(a, b) for a, b in zip(out[0][1], out[1][1]))
    assert torch.equal(out[0][0], out[1][0])


# ----------------------------------------------------------------------------- grouped-query attention
def test_grouped_query_attention_prefill_fp32():
    """Fewer key/value heads than query heads (2 of 4, then 1 of 4): the whole pruned prefill against the
    oracle on the generic fp32 kernels, varlen batch included; caches hold key/value heads only."""
    for kvh in (2, 1):
        shape = synth.TINY.with_layers(3).with_kv_heads(kvh)
        run_model_case(shape, ((1, 6000), (2, 3000)), [90, 1, 47], torch.float32, seed=30 + kvh)


def test_grouped_query_attention_prefill_bf16_tensor_cores():
    """head_dim 128, 4 query heads on 2 key/value heads: QKV projection with RoPE and the cache write in its
    epilogue over [q | k | v] sections of different widths, tcgen05 attention reading key/value head h // 2."""
    shape = synth.SMALL.with_kv_heads(2)
    run_model_case(shape, ((1, 7000), (2, 5000), (3, 3000)), [300], torch.bfloat16, seed=33)
    run_model_case(shape.with_layers(3), ((1, 6000), (2, 3000)), [200, 65, 1, 131], torch.bfloat16, seed=34)


def test_grouped_query_attention_wide_shape_bf16():
    """Two layers of a 7B-class grouped shape (d=4096, 32 query heads on 8 key/value heads, ffn 11008), 700-token
    prompt with a cut: the widths at which the fused projection is 6144 columns wide and the caches 1024."""
    shape = synth.ModelShape(n_layers=2, d_model=4096, n_heads=32, head_dim=128, d_ffn=11008, vocab=4096,
                             n_kv_heads=8)
    run_model_case(shape, ((1, 5000),), [700], torch.bfloat16, seed=35, perturb=False)


# ----------------------------------------------------------------------------- e4m3 projections end to end
def test_fp8_projections_prefill_small_model():
    """The four projections of every layer on e4m3 operands (per-row activation scales, per-matrix weight
    scales), everything else in bf16: pruned prefill against the oracle run in the same mode, on the same
    de-quantised weights; kept sets, scores, hidden states, caches, Aux rows and logits."""
    shape = synth.SMALL.with_fp8()
    run_model_case(shape, ((1, 7000), (2, 5000), (3, 3000)), [300], torch.bfloat16, seed=41)
    run_model_case(shape.with_layers(3).with_kv_heads(2), ((1, 6000), (2, 3000)), [200, 65, 9, 131], torch.bfloat16, seed=42)


def test_fp8_projections_wide_shape_and_against_bf16():
    """Two layers at the 7B widths, 1500-token prompt, one cut, against the oracle in the same mode."""
    shape = synth.LLAMA7B.with_layers(2).with_fp8()
    run_model_case(shape, ((1, 5000),), [1500], torch.bfloat16, seed=43, perturb=False)
