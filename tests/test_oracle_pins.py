"""Pins for the CPU oracle: library cross-checks, closed forms, brute force, invariants.

Nothing here touches the CUDA path.  Each pin is chosen so that a plausible slip in the
oracle (a dropped term, a transposed operand, the wrong attention row, a wrong RoPE
pairing, an off-by-one in the keep count) makes at least one of them fail.
"""
import os

import numpy as np
import pytest
import torch

import lazyllm_oracle as O
from paper_2407_14057_b200 import synth
from helpers import weights_to_np, to_np, rel_err

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")

MINI = synth.ModelShape(n_layers=3, d_model=64, n_heads=4, head_dim=16, d_ffn=176, vocab=128)


def mini_weights(seed=11, shape=MINI, std=0.2):
    W = synth.make_weights(shape, seed, bf16=False, std=std)
    synth.perturb_gains(W, seed + 1)
    return W


# ----------------------------------------------------------------------------- library pin
def _hf_model(shape, W):
    from transformers import LlamaConfig, LlamaForCausalLM
    cfg = LlamaConfig(vocab_size=shape.vocab, hidden_size=shape.d_model,
                      intermediate_size=shape.d_ffn, num_hidden_layers=shape.n_layers,
                      num_attention_heads=shape.n_heads, num_key_value_heads=shape.kv_heads,
                      head_dim=shape.head_dim, rms_norm_eps=shape.rms_eps,
                      rope_theta=shape.rope_theta, attention_bias=False, mlp_bias=False,
                      tie_word_embeddings=False, attn_implementation="eager",
                      max_position_embeddings=1024)
    m = LlamaForCausalLM(cfg).double().eval()
    d = shape.d_model
    sd = {"model.embed_tokens.weight": W["tok_embed"], "model.norm.weight": W["g_final"],
          "lm_head.weight": W["w_lm_head"]}
    for l, lw in enumerate(W["layers"]):
        p = f"model.layers.{l}."
        sd[p + "self_attn.q_proj.weight"] = lw["w_qkv"][:d]
        dkv = shape.kv_heads * shape.head_dim
        sd[p + "self_attn.k_proj.weight"] = lw["w_qkv"][d:d + dkv]
        sd[p + "self_attn.v_proj.weight"] = lw["w_qkv"][d + dkv:]
        sd[p + "self_attn.o_proj.weight"] = lw["w_o"]
        sd[p + "mlp.gate_proj.weight"] = lw["w_gate"]
        sd[p + "mlp.up_proj.weight"] = lw["w_up"]
        sd[p + "mlp.down_proj.weight"] = lw["w_down"]
        sd[p + "input_layernorm.weight"] = lw["g_attn"]
        sd[p + "post_attention_layernorm.weight"] = lw["g_mlp"]
    missing = m.load_state_dict({k: v.double() for k, v in sd.items()}, strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k]
    return m


def test_full_keep_matches_library_llama():
    """100 % keep == standard prefill: logits, per-layer hidden states and the head-mean of the
    last attention row agree with the transformers Llama implementation run in fp64 (which still
    evaluates its rotary cos/sin tables in fp32: hence 1e-5, not 1e-12; a convention slip is O(1))."""
    W = mini_weights()
    ids = synth.make_prompt(MINI.vocab, 37, seed=3)
    m = _hf_model(MINI, W)
    with torch.no_grad():
        out = m(ids.long()[None], output_attentions=True, output_hidden_states=True)
    st = O.prefill(MINI, weights_to_np(W), to_np(ids), schedule=())
    assert rel_err(st.logits, out.logits[0, -1].numpy()) < 1e-5
    for l in range(MINI.n_layers):
        ref_s = out.attentions[l][0, :, -1, :].mean(dim=0).numpy()
        assert np.max(np.abs(st.scores[l] - ref_s)) < 1e-6
        if l + 1 < MINI.n_layers:  # the library applies the final norm to its last entry
            assert rel_err(st.hidden_out[l], out.hidden_states[l + 1][0].numpy()) < 1e-5


def test_grouped_query_attention_matches_library_llama():
    """Fewer key/value heads than query heads (query head h reads key/value head h // group): logits, hidden
    states, the head-mean last attention row and greedy decode against the library's Llama with
    num_key_value_heads = 2 of 4 heads and 1 of 4 heads."""
    for kvh in (2, 1):
        shape = MINI.with_kv_heads(kvh)
        W = mini_weights(seed=40 + kvh, shape=shape)
        assert W["layers"][0]["w_qkv"].shape[0] == shape.d_model + 2 * kvh * shape.head_dim
        ids = synth.make_prompt(shape.vocab, 29, seed=6)
        m = _hf_model(shape, W)
        with torch.no_grad():
            out = m(ids.long()[None], output_attentions=True, output_hidden_states=True)
            gen = m.generate(ids.long()[None], max_new_tokens=3, do_sample=False, use_cache=True)
        Wn = weights_to_np(W)
        st = O.prefill(shape, Wn, to_np(ids), schedule=())
        assert rel_err(st.logits, out.logits[0, -1].numpy()) < 1e-5
        for l in range(shape.n_layers):
            ref_s = out.attentions[l][0, :, -1, :].mean(dim=0).numpy()
            assert np.max(np.abs(st.scores[l] - ref_s)) < 1e-6
            assert st.layers[l].kv[0][0].shape == (kvh, shape.head_dim)      # the cache holds kv heads only
        got = [O.greedy(st.logits)]
        for _ in range(2):
            got.append(O.greedy(O.decode_step(shape, Wn, st, got[-1])))
        assert got == gen[0, ids.shape[0]:].tolist()
        # pruning on top: invariants of the pruned run hold with grouped heads as well
        pr = O.prefill(shape, Wn, to_np(ids), ((1, 6000), (2, 3000)))
        assert [len(pr.kept_pos[e]) for e in (1, 2)] == [18, 9] and abs(pr.scores[2].sum() - 1) < 1e-12


def test_decode_full_keep_matches_library_greedy():
    """With nothing pruned, prefill + decode steps reproduce the library's greedy generation."""
    W = mini_weights(seed=21)
    Wn = weights_to_np(W)
    ids = synth.make_prompt(MINI.vocab, 19, seed=5)
    m = _hf_model(MINI, W)
    with torch.no_grad():
        gen = m.generate(ids.long()[None], max_new_tokens=5, do_sample=False, use_cache=True)
    ref = gen[0, ids.shape[0]:].tolist()
    st = O.prefill(MINI, Wn, to_np(ids), schedule=((1, 10000), (2, 10000)))
    got = [O.greedy(st.logits)]
    for _ in range(4):
        got.append(O.greedy(O.decode_step(MINI, Wn, st, got[-1])))
    assert got == ref


# ----------------------------------------------------------------------------- Eq. 1
def test_score_is_a_probability_vector():
    W = weights_to_np(mini_weights(seed=2))
    ids = to_np(synth.make_prompt(MINI.vocab, 50, seed=1))
    st = O.prefill(MINI, W, ids, schedule=((1, 6000), (2, 3000)))
    for s in st.scores:
        assert np.all(s >= 0)
        assert abs(np.sum(s) - 1.0) < 1e-12


def test_score_single_token_closed_form():
    W = weights_to_np(mini_weights(seed=2))
    st = O.prefill(MINI, W, np.array([5]), schedule=())
    for s in st.scores:
        assert s.shape == (1,) and s[0] == 1.0


def test_score_uniform_when_queries_vanish():
    """Zero query projection => every visible key gets the same logit => s_j = 1/n."""
    Wt = mini_weights(seed=4)
    for lw in Wt["layers"]:
        lw["w_qkv"][:MINI.d_model] = 0
    st = O.prefill(MINI, weights_to_np(Wt), to_np(synth.make_prompt(MINI.vocab, 23, seed=1)), ())
    for s in st.scores:
        assert np.max(np.abs(s - 1.0 / 23)) < 1e-15


def test_score_is_last_row_not_last_column():
    """The last COLUMN of a causal attention matrix is zero except its final entry; Eq. 1 under
    the adopted reading spreads mass over earlier tokens."""
    W = weights_to_np(mini_weights(seed=6))
    st = O.prefill(MINI, W, to_np(synth.make_prompt(MINI.vocab, 16, seed=2)), ())
    assert np.count_nonzero(st.scores[0][:-1] > 1e-6) >= 8


def test_attention_probs_two_token_closed_form():
    q = np.array([[1.0, 0.0], [2.0, 0.0]])
    k = np.array([[3.0, 0.0], [1.0, 0.0]])
    A = O.attention_probs(q, k, np.array([0, 1]), np.array([0, 1]))
    assert np.allclose(A[0], [1.0, 0.0])
    a, b = 2 * 3 / np.sqrt(2), 2 * 1 / np.sqrt(2)
    assert np.allclose(A[1], np.exp([a, b]) / np.sum(np.exp([a, b])))


def test_rope_rotation_closed_form():
    """dh=4: pairs (0,2) and (1,3); frequencies 1 and theta^-1/2; a pure rotation."""
    x = np.array([[[1.0, 2.0, 0.0, 0.0]]])
    y = O.rope(x, np.array([3]), 100.0)[0, 0]
    assert np.allclose(y, [np.cos(3.0), 2 * np.cos(0.3), np.sin(3.0), 2 * np.sin(0.3)])
    z = O.rope(np.random.default_rng(0).normal(size=(5, 2, 8)), np.arange(5), 1e4)
    assert np.allclose(np.linalg.norm(z, axis=-1),
                       np.linalg.norm(np.random.default_rng(0).normal(size=(5, 2, 8)), axis=-1))


def test_rope_relative_position_property():
    """<rope(q,m), rope(k,n)> depends on m-n only."""
    rng = np.random.default_rng(1)
    q, k = rng.normal(size=(1, 1, 16)), rng.normal(size=(1, 1, 16))
    d1 = np.sum(O.rope(q, np.array([7]), 1e4) * O.rope(k, np.array([3]), 1e4))
    d2 = np.sum(O.rope(q, np.array([104]), 1e4) * O.rope(k, np.array([100]), 1e4))
    assert abs(d1 - d2) < 1e-9


# ----------------------------------------------------------------------------- selection
def _rank_count_select(s, n_keep, forced):
    """Independent O(n^2) formulation: a candidate's rank is the number of candidates that beat
    it (greater score, or equal score and lower index); forced candidate has rank -1."""
    n = len(s)
    keep = []
    for i in range(n):
        if i == forced:
            keep.append(i)
            continue
        rank = sum(1 for j in range(n) if j != forced and (s[j] > s[i] or (s[j] == s[i] and j < i)))
        if rank < n_keep - 1:
            keep.append(i)
    return keep


def _load_select_cases():
    cases = []
    with open(os.path.join(GOLDEN, "select_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            a, b, c, d = [t.strip() for t in line.split("|")]
            cases.append((np.array([float(v) for v in a.split()]), int(b),
                          [int(v) for v in c.split()], [int(v) for v in d.split()]))
    return cases


def test_select_hand_worked_cases():
    cases = _load_select_cases()
    assert len(cases) >= 12
    for s, n_keep, kept, dropped in cases:
        k, d = O.select_top(s, n_keep, len(s) - 1)
        assert k.tolist() == kept and d.tolist() == dropped, (s, n_keep)


@pytest.mark.parametrize("kind", ["random", "uniform", "zeros", "duplicates", "lognormal"])
@pytest.mark.parametrize("n", [1, 2, 5, 127, 300])
def test_select_matches_rank_count_brute_force(kind, n):
    s = synth.make_scores(n, kind, seed=n).numpy()
    for n_keep in sorted({1, max(1, n // 3), max(1, (n * 6 + 9) // 10), n}):
        keep, drop = O.select_top(s, n_keep, n - 1)
        assert keep.tolist() == _rank_count_select(s, n_keep, n - 1)
        assert len(keep) == n_keep and (n - 1) in keep
        assert sorted(keep.tolist() + drop.tolist()) == list(range(n))
        assert np.all(np.diff(keep) > 0) and np.all(np.diff(drop) > 0)
        free = [i for i in keep if i != n - 1]
        if free and len(drop):
            assert min(s[free]) >= max(s[drop])


def test_select_threshold_is_the_lower_percentile_with_ties_kept():
    rng = np.random.default_rng(5)
    for n in (1, 2, 7, 64, 501):
        s = rng.random(n).astype(np.float32)
        for bp in (0, 1, 2500, 3000, 5000, 9999):
            keep, drop = O.select_threshold(s, bp)
            tau = np.percentile(s, bp / 100.0, method="lower")            # library pin for the threshold
            want = sorted(set(np.nonzero(s >= tau)[0].tolist()) | {n - 1})
            assert keep.tolist() == want
            assert sorted(keep.tolist() + drop.tolist()) == list(range(n))
            assert len(keep) >= n - ((n - 1) * bp) // 10000                # at least the rank says; more on ties
    # hand-worked: scores 5 1 3 3 2, 50th percentile (lower) = sorted[2] = 3 -> keep rows 0, 2, 3 and the last
    keep, drop = O.select_threshold(np.array([5, 1, 3, 3, 2], dtype=np.float32), 5000)
    assert keep.tolist() == [0, 2, 3, 4] and drop.tolist() == [1]
    # all equal: nothing can be below the threshold
    keep, drop = O.select_threshold(np.ones(9, dtype=np.float32), 9000)
    assert keep.tolist() == list(range(9)) and drop.tolist() == []
    # without ties the count agrees with the count-based form at the matching count
    s = rng.permutation(200).astype(np.float32)
    keep, _ = O.select_threshold(s, 4000)
    k2, _ = O.select_top(s, len(keep), len(s) - 1)     # the last token counts toward the kept set there too
    assert keep.tolist() == sorted(k2.tolist())
    with pytest.raises(ValueError):
        O.select_threshold(s, 10000)


def test_keep_count_worked_values():
    with open(os.path.join(GOLDEN, "keep_counts.txt")) as f:
        rows = [l for l in f if l.strip() and not l.startswith("#")]
    assert len(rows) >= 10
    for line in rows:
        N, bp, want = [int(t) for t in line.split("|")]
        assert O.keep_count(N, bp, N) == want
    assert O.keep_count(100, 7000, 50) == 50       # clamped to the rows present


# ----------------------------------------------------------------------------- pruned prefill
def _pruned_and_full(seed=8, n=61, schedule=((1, 7000), (2, 4000))):
    W = weights_to_np(mini_weights(seed=seed))
    ids = to_np(synth.make_prompt(MINI.vocab, n, seed=seed))
    return W, ids, O.prefill(MINI, W, ids, schedule), O.prefill(MINI, W, ids, ())


def test_no_approximation_before_first_cut():
    W, ids, pr, full = _pruned_and_full()
    assert np.array_equal(pr.scores[0], full.scores[0])
    assert np.array_equal(pr.hidden_after_attn[0], full.hidden_after_attn[0])
    kept = pr.kept_pos[1]
    assert np.array_equal(pr.hidden_out[0], full.hidden_out[0][kept])   # MLP is row-wise


def test_aux_cache_holds_dropped_rows_of_first_cut_exactly():
    W, ids, pr, full = _pruned_and_full()
    dropped = pr.dropped_pos[1]
    assert len(dropped) == 61 - O.keep_count(61, 7000, 61)
    assert sorted(pr.layers[0].aux.keys()) == dropped.tolist()
    for p in dropped:
        assert np.array_equal(pr.layers[0].aux[int(p)], full.hidden_after_attn[0][p])
    assert pr.layers[2].aux == {}


def test_subset_property_and_cache_membership():
    W, ids, pr, full = _pruned_and_full()
    c = [set(l.kv.keys()) for l in pr.layers]
    assert c[0] == set(range(61))
    assert c[2] <= c[1] <= c[0]
    assert len(c[1]) == O.keep_count(61, 7000, 61) and len(c[2]) == O.keep_count(61, 4000, 61)
    for l in range(2):
        assert set(pr.layers[l].aux.keys()) == c[l] - c[l + 1]
    assert all(60 in s for s in c)                      # last token never pruned
    assert all(v == 1 for v in pr.compute_count.values())


def test_keep_one_makes_later_attention_the_identity_on_v():
    W = weights_to_np(mini_weights(seed=9))
    ids = to_np(synth.make_prompt(MINI.vocab, 12, seed=9))
    st = O.prefill(MINI, W, ids, ((1, 1),))
    assert st.kept_pos[1].tolist() == [11]
    for l in (1, 2):
        v = st.layers[l].kv[11][1].reshape(-1)
        delta = st.hidden_after_attn[l][0] - st.hidden_out[l - 1][0]
        assert np.allclose(delta, v @ W["layers"][l]["w_o"].astype(np.float64).T, atol=1e-13)
        assert st.scores[l].tolist() == [1.0]


def test_layer_step_chain_is_bitwise_the_prefill():
    """`layer_step` is the loop body of `prefill`: chaining it over the layers, with the kept sets of
    a prefill run, reproduces that run exactly (so per-layer checks against it mean the same)."""
    W, ids, pr, full = _pruned_and_full()
    x = np.asarray(W["tok_embed"], dtype=np.float64)[ids]
    pos = np.arange(len(ids))
    for l in range(MINI.n_layers):
        r = O.layer_step(MINI, W["layers"][l], x, pos, keep_pos=pr.kept_pos.get(l + 1))
        assert np.array_equal(r["scores"], pr.scores[l])
        assert np.array_equal(r["hidden_attn"], pr.hidden_after_attn[l])
        assert np.array_equal(r["hidden_out"], pr.hidden_out[l])
        assert sorted(pr.layers[l].aux.keys()) == r["aux_pos"].tolist()
        x, pos = r["hidden_out"], r["pos_out"]
    assert np.array_equal(O.lm_head(MINI, W, x[-1]), pr.logits)


def test_forced_keep_replays_the_same_run():
    W, ids, pr, full = _pruned_and_full()
    again = O.prefill(MINI, W, ids, ((1, 7000), (2, 4000)), forced_keep=dict(pr.kept_pos))
    assert np.array_equal(again.logits, pr.logits)
    other = {1: np.arange(20, 61), 2: np.arange(40, 61)}
    alt = O.prefill(MINI, W, ids, ((1, 7000), (2, 4000)), forced_keep=other)
    assert alt.kept_pos[2].tolist() == list(range(40, 61))


def test_full_keep_schedule_is_bitwise_standard_prefill():
    W, ids, pr, full = _pruned_and_full()
    same = O.prefill(MINI, W, ids, ((1, 10000), (2, 10000)))
    assert np.array_equal(same.logits, full.logits)
    assert all(l.aux == {} for l in same.layers)


def test_bad_schedules_are_rejected():
    W = weights_to_np(mini_weights())
    for bad in [((0, 5000),), ((3, 5000),), ((2, 5000), (1, 4000)), ((1, 5000), (2, 6000)),
                ((1, 0),), ((1, 10001),)]:
        with pytest.raises(ValueError):
            O.prefill(MINI, W, np.arange(8), bad)


# ----------------------------------------------------------------------------- revive
def _recompute_token(cfg, W, st, t, upto_layer):
    """Hidden state of token t after the attention of ``upto_layer``, recomputed alone from the
    embedding against the cached K/V rows with position <= t (textbook KV-cache forward)."""
    x = np.asarray(W["tok_embed"], dtype=np.float64)[t[1]][None]
    pos = np.array([t[0]])
    for l in range(upto_layer + 1):
        lw = W["layers"][l]
        q, k, v = O._layer_qkv(cfg, lw, x, pos)
        ctx = np.array(sorted(p for p in st.layers[l].kv if p <= t[0]))
        kc, vc = st.layers[l].rows(ctx)
        o, _ = O.attend(q, kc, vc, pos, ctx, 0)
        x = x + o @ np.asarray(lw["w_o"], dtype=np.float64).T
        if l < upto_layer:
            x = x + O.mlp(cfg, lw, x)
    return x[0]


def test_revived_token_matches_its_recomputed_hidden_state():
    W, ids, pr, full = _pruned_and_full(seed=13, n=47)
    for layer_entered in (1, 2):
        dropped = pr.dropped_pos[layer_entered]
        assert len(dropped) > 0
        rows = O.revive(pr, layer_entered - 1, dropped)
        for i, p in enumerate(dropped[:6]):
            ref = _recompute_token(MINI, W, pr, (int(p), int(ids[p])), layer_entered - 1)
            assert np.max(np.abs(rows[i] - ref)) < 1e-12
    with pytest.raises(KeyError):
        O.revive(pr, 0, [int(pr.kept_pos[1][0])])


# ----------------------------------------------------------------------------- decode
def test_decode_full_keep_equals_prefill_of_longer_prompt():
    W = weights_to_np(mini_weights(seed=15))
    ids = to_np(synth.make_prompt(MINI.vocab, 30, seed=15))
    st = O.prefill(MINI, W, ids[:26], ((1, 10000),))
    for t in range(26, 30):
        logits = O.decode_step(MINI, W, st, int(ids[t]))
        ref = O.prefill(MINI, W, ids[:t + 1], ())
        assert rel_err(logits, ref.logits) < 1e-12
        assert all(len(v) == 0 for v in st.revived_pos.values())


def test_decode_invariants_with_pruning():
    shape = MINI.with_layers(5)
    W = weights_to_np(mini_weights(seed=17, shape=shape))
    ids = to_np(synth.make_prompt(shape.vocab, 40, seed=17))
    schedule = ((1, 7000), (2, 5000), (4, 3000))
    st = O.prefill(shape, W, ids, schedule)
    tok = O.greedy(st.logits)
    revived_total = 0
    for step in range(8):
        logits = O.decode_step(shape, W, st, tok)
        p = 40 + step
        tok = O.greedy(logits)
        c = [set(l.kv.keys()) for l in st.layers]
        for l in range(shape.n_layers - 1):
            assert c[l + 1] <= c[l]                                   # subset property
            assert set(st.layers[l].aux.keys()) == c[l] - c[l + 1]      # Aux = C_l \ C_{l+1}
            if (l + 1) not in dict(schedule):
                assert c[l + 1] == c[l]
        assert all(p in s for s in c)                                 # current token everywhere
        assert c[0] == set(range(p + 1))
        assert all(v == 1 for v in st.compute_count.values())         # at most once per layer
        for e, bp in schedule:
            assert len(st.kept_pos[e]) == O.keep_count(p + 1, bp, p + 1) or \
                len(st.kept_pos[e]) <= O.keep_count(p + 1, bp, p + 1)
            assert p in st.kept_pos[e]
        for s in st.scores:
            assert abs(np.sum(s) - 1) < 1e-12
        revived_total += sum(len(v) for v in st.revived_pos.values())
    assert revived_total > 0          # the case exercises revival
    frac = O.tokens_computed_fraction(st, 40)
    assert frac[0] == 1.0 and all(0 < f <= 1.0 for f in frac)
    assert all(frac[l + 1] <= frac[l] for l in range(shape.n_layers - 1))
    # exact values, counted independently from the caches: prompt positions are 0..39, generated
    # tokens (positions >= 40) must not count, position 39 must
    for l, c in enumerate(st.layers):
        assert frac[l] == len(set(c.kv.keys()) & set(range(40))) / 40.0


def test_tokens_computed_fraction_hand_worked():
    """Right after a prefill of 10 tokens with keep 70 % entering layer 1 and 30 % entering layer 2, the
    fractions are 10/10, 7/10, 3/10 by the keep counts alone; a decode step adds position 10, which is
    not a prompt token, and revives prompt tokens only into layers that already count them or not."""
    shape = MINI
    W = weights_to_np(mini_weights(seed=23))
    ids = to_np(synth.make_prompt(shape.vocab, 10, seed=23))
    st = O.prefill(shape, W, ids, ((1, 7000), (2, 3000)))
    assert O.tokens_computed_fraction(st, 10) == [1.0, 0.7, 0.3] + [0.3] * (shape.n_layers - 3)
    # a boundary case of the prompt/generated split: with n_prompt = 9, position 9 is not counted
    assert O.tokens_computed_fraction(st, 9)[0] == 1.0
    assert O.tokens_computed_fraction(st, 11)[0] == 10.0 / 11.0


def test_decode_revived_row_feeds_deferred_mlp():
    """A token revived into layer e runs the MLP of layer e-1 first: its K/V at layer e equals
    what a direct evaluation from the Aux row gives."""
    shape = MINI
    W = weights_to_np(mini_weights(seed=19))
    ids = to_np(synth.make_prompt(shape.vocab, 24, seed=19))
    st = O.prefill(shape, W, ids, ((1, 5000),))
    aux_before = {p: x.copy() for p, x in st.layers[0].aux.items()}
    forced = {1: np.arange(24)}                           # select everything: all dropped revive
    O.decode_step(shape, W, st, 7, forced_keep=forced)
    assert sorted(st.revived_pos[1].tolist()) == sorted(aux_before.keys())
    assert st.layers[0].aux == {}
    p0 = sorted(aux_before.keys())[0]
    x = aux_before[p0][None]
    x = x + O.mlp(shape, W["layers"][0], x)
    _, k, v = O._layer_qkv(shape, W["layers"][1], x, np.array([p0]))
    assert np.allclose(st.layers[1].kv[p0][0], k[0], atol=1e-13)
    assert np.allclose(st.layers[1].kv[p0][1], v[0], atol=1e-13)


# ------------------------------------------------------- the cut after the whole layer ("post_layer")
def test_post_layer_aux_point_prefill_same_tokens_same_values_aux_is_layer_output():
    """The MLP is row-wise, so cutting after the whole scoring layer instead of before its MLP changes
    nothing downstream: same kept sets, same hidden states of kept rows, same logits.  Only the Aux Cache
    differs, and by exactly that layer's MLP (with its residual) applied to the pre-MLP rows."""
    shape = MINI.with_layers(5)
    W = weights_to_np(mini_weights(seed=23, shape=shape))
    ids = to_np(synth.make_prompt(shape.vocab, 47, seed=23))
    schedule = ((1, 7000), (3, 4000), (4, 2500))
    a = O.prefill(shape, W, ids, schedule)
    b = O.prefill(shape, W, ids, schedule, aux_point="post_layer")
    for e, _ in schedule:
        assert np.array_equal(a.kept_pos[e], b.kept_pos[e])
        assert np.array_equal(a.dropped_pos[e], b.dropped_pos[e])
    for l in range(shape.n_layers):
        assert np.allclose(a.hidden_out[l], b.hidden_out[l], rtol=0, atol=1e-12)
        assert set(a.layers[l].kv) == set(b.layers[l].kv)
        assert set(a.layers[l].aux) == set(b.layers[l].aux)
        for pos_, xa in a.layers[l].aux.items():
            want = xa[None] + O.mlp(shape, W["layers"][l], xa[None])
            assert np.allclose(b.layers[l].aux[pos_], want[0], rtol=0, atol=1e-12)
    assert np.allclose(a.logits, b.logits, rtol=0, atol=1e-11)
    with pytest.raises(ValueError):
        O.prefill(shape, W, ids, schedule, aux_point="mid_layer")


def test_post_layer_aux_point_decode_same_logits_selection_and_revivals():
    """Through decode steps with revival the two cut points stay equivalent: same logits, same re-selected
    contexts, same revived tokens, each token still computed at most once per layer, Aux = C_l minus
    C_{l+1}; and a revived token's K/V in the next layer comes straight from its Aux row (no deferred MLP)."""
    shape = MINI.with_layers(5)
    W = weights_to_np(mini_weights(seed=29, shape=shape))
    ids = to_np(synth.make_prompt(shape.vocab, 40, seed=29))
    schedule = ((1, 7000), (2, 5000), (4, 3000))
    a = O.prefill(shape, W, ids, schedule)
    b = O.prefill(shape, W, ids, schedule, aux_point="post_layer")
    tok = O.greedy(a.logits)
    revived_total = 0
    for step in range(8):
        aux_b_before = [{p_: x.copy() for p_, x in l.aux.items()} for l in b.layers]
        la = O.decode_step(shape, W, a, tok)
        lb = O.decode_step(shape, W, b, tok)
        assert np.allclose(la, lb, rtol=0, atol=1e-10)
        for e, _ in schedule:
            assert np.array_equal(a.kept_pos[e], b.kept_pos[e])
            assert np.array_equal(np.sort(a.revived_pos[e]), np.sort(b.revived_pos[e]))
            for r in b.revived_pos[e]:                                  # straight from the Aux row
                x = aux_b_before[e - 1][int(r)][None]
                _, k, v = O._layer_qkv(shape, W["layers"][e], x, np.array([int(r)]))
                assert np.allclose(b.layers[e].kv[int(r)][0], k[0], atol=1e-13)
                assert np.allclose(b.layers[e].kv[int(r)][1], v[0], atol=1e-13)
            revived_total += len(b.revived_pos[e])
        c = [set(l.kv.keys()) for l in b.layers]
        for l in range(shape.n_layers - 1):
            assert c[l + 1] <= c[l]
            assert set(b.layers[l].aux.keys()) == c[l] - c[l + 1]
        assert all(v == 1 for v in b.compute_count.values())
        tok = O.greedy(la)
    assert revived_total > 0


def test_prune_op_agrees_with_prefill_first_layer():
    shape = MINI
    W = weights_to_np(mini_weights(seed=23))
    ids = to_np(synth.make_prompt(shape.vocab, 33, seed=23))
    st = O.prefill(shape, W, ids, ((1, 6000),))
    x0 = np.asarray(W["tok_embed"], dtype=np.float64)[ids]
    r = O.prune_op(shape, W["layers"][0], x0, np.arange(33), 6000)
    assert np.array_equal(r["scores"], st.scores[0])
    assert np.array_equal(r["pos_kept"], st.kept_pos[1])
    assert np.array_equal(r["hidden_attn"], st.hidden_after_attn[0])
    assert sorted(st.layers[0].aux.keys()) == r["aux_pos"].tolist()
    assert np.array_equal(r["k_kept"][0], st.layers[0].kv[int(r["pos_kept"][0])][0])


# ----------------------------------------------------------------------------- threshold reading, ties kept
def test_select_ties_kept_hand_worked():
    """Worked by hand from the definition: tau = the n_keep-th largest score with the forced (last) token
    counted as the largest; pruned iff score < tau."""
    s = np.array([0.30, 0.10, 0.10, 0.05, 0.10, 0.02], dtype=np.float32)   # forced = index 5
    # n_keep = 3: places go to {5 (forced), 0.30, 0.10}; tau = 0.10; the three 0.10s all survive
    keep, drop = O.select_ties_kept(s, 3, 5)
    assert keep.tolist() == [0, 1, 2, 4, 5] and drop.tolist() == [3]
    # the count form keeps exactly three, the tie going to the lower index
    k2, d2 = O.select_top(s, 3, 5)
    assert k2.tolist() == [0, 1, 5] and d2.tolist() == [2, 3, 4]
    # n_keep = 2: tau = 0.30, no tie: both forms agree
    assert O.select_ties_kept(s, 2, 5)[0].tolist() == O.select_top(s, 2, 5)[0].tolist() == [0, 5]
    # n_keep = 1: only the forced token
    assert O.select_ties_kept(s, 1, 5)[0].tolist() == [5]
    # everything equal: nothing is smaller than tau, nothing is pruned
    u = np.full(7, 1.0 / 7, dtype=np.float32)
    assert O.select_ties_kept(u, 3, 6)[0].tolist() == list(range(7))
    # the forced token's own score does not move the threshold (here it would be the largest)
    t = np.array([0.1, 0.2, 0.3, 0.9], dtype=np.float32)
    assert O.select_ties_kept(t, 2, 3)[0].tolist() == [2, 3]


def test_select_ties_kept_equals_count_form_without_ties_and_brute_force_with():
    rng = np.random.default_rng(31)
    for n in (1, 2, 5, 64, 257):
        s = rng.permutation(n).astype(np.float32)          # all distinct
        for n_keep in sorted({1, max(1, n // 3), n}):
            a = O.select_ties_kept(s, n_keep, n - 1)
            b = O.select_top(s, n_keep, n - 1)
            assert a[0].tolist() == b[0].tolist() and a[1].tolist() == b[1].tolist()
    for _ in range(50):                                     # few levels: ties everywhere
        n = int(rng.integers(2, 40))
        s = rng.integers(0, 4, n).astype(np.float32)
        n_keep = int(rng.integers(1, n + 1))
        keep, drop = O.select_ties_kept(s, n_keep, n - 1)
        k_top, _ = O.select_top(s, n_keep, n - 1)
        assert set(k_top.tolist()) <= set(keep.tolist()) and len(keep) >= n_keep     # a superset of the count form
        if len(drop):
            tau = min(float(s[i]) for i in keep if i != n - 1) if len(keep) > 1 else np.inf
            assert all(float(s[i]) < tau for i in drop)                              # pruned iff strictly smaller
        assert sorted(keep.tolist() + drop.tolist()) == list(range(n))


def test_threshold_prefill_equals_count_prefill_without_ties_and_keeps_all_ties():
    """Generic inputs have no ties: both readings give the same run.  A layer whose query projection is zero
    attends uniformly (closed form s_j = 1/n), every score ties, and the threshold reading prunes nothing
    there while the count reading prunes down to the schedule."""
    shape = MINI
    W = weights_to_np(mini_weights(seed=29))
    ids = to_np(synth.make_prompt(shape.vocab, 30, seed=29))
    sched = ((1, 6000), (2, 3000))
    a = O.prefill(shape, W, ids, sched, selection="count")
    b = O.prefill(shape, W, ids, sched, selection="threshold")
    assert all(np.array_equal(a.kept_pos[e], b.kept_pos[e]) for e, _ in sched)
    assert np.array_equal(a.logits, b.logits)
    d = shape.d_model
    W["layers"][0] = dict(W["layers"][0])
    wq = np.array(W["layers"][0]["w_qkv"], copy=True)
    wq[:d] = 0.0                                           # q = 0 in layer 0: uniform attention rows
    W["layers"][0]["w_qkv"] = wq
    c = O.prefill(shape, W, ids, sched, selection="count")
    t = O.prefill(shape, W, ids, sched, selection="threshold")
    assert np.allclose(t.scores[0], 1.0 / 30) and len(np.unique(t.scores[0])) == 1
    assert len(c.kept_pos[1]) == 18 and len(t.kept_pos[1]) == 30          # nothing is smaller than tau
    assert len(t.kept_pos[2]) == O.keep_count(30, 3000, 30) == 9           # the next cut has no ties again
    assert len(t.layers[0].aux) == 0 and len(c.layers[0].aux) == 12
    # decode keeps using the state's reading
    assert t.selection == "threshold"
    O.decode_step(shape, W, t, O.greedy(t.logits))


# ----------------------------------------------------------------------------- e4m3 projections
def test_round_e4m3_hand_worked_and_against_the_library_cast():
    """e4m3: 3 mantissa bits, so 8 steps per binade; ties go to the even mantissa; largest value 448;
    below 2^-6 the step stays 2^-9."""
    x = np.array([0.3, 17.0, 19.0, 21.0, 448.0, 500.0, -1000.0, 1.0625, 1.1875, 2.0 ** -7, 2.0 ** -10, 0.0, -0.3],
                 dtype=np.float32)
    want = [0.3125, 16.0, 20.0, 20.0, 448.0, 448.0, -448.0, 1.0, 1.25, 2.0 ** -7, 2.0 ** -9 * 0.0, 0.0, -0.3125]
    # 17 lies between 16 and 18: tie, even mantissa 000 -> 16; 19 between 18 (001) and 20 (010) -> 20;
    # 21 between 20 and 22 (011): tie -> 20; 1.0625 between 1.0 and 1.125 -> 1.0; 1.1875 between 1.125 (001)
    # and 1.25 (010) -> 1.25; 2^-10 is half a subnormal step: tie between 0 and 2^-9 -> 0 (even)
    assert O.round_e4m3(x).tolist() == want
    g = torch.Generator().manual_seed(5)
    r = (torch.randn(20000, generator=g) * torch.logspace(-4, 2.5, 20000)).float()
    r = r.clamp(-448, 448)
    lib = r.to(torch.float8_e4m3fn).float().numpy()
    assert np.array_equal(O.round_e4m3(r.numpy()), lib)


def test_quant_rows_e4m3_properties():
    rng = np.random.default_rng(9)
    x = (rng.standard_normal((7, 96)) * rng.uniform(0.01, 30, (7, 1))).astype(np.float32)
    x[3] = 0.0
    codes, scale = O.quant_rows_e4m3(x)
    assert scale[3] == 1.0 and np.all(codes[3] == 0)
    for r in (0, 1, 2, 4, 5, 6):
        assert scale[r] == np.float32(np.abs(x[r]).max()) / np.float32(448.0)
        assert np.abs(codes[r]).max() == 448.0                       # the largest element lands on the top code
        assert np.array_equal(codes[r], O.round_e4m3(x[r] / scale[r]))
        assert np.max(np.abs(codes[r] * scale[r] - x[r])) <= np.abs(x[r]).max() / 448.0 * 16.0 + 1e-12   # half a top-binade step
        rel = np.abs(codes[r] * scale[r] - x[r]) / np.abs(x[r]).clip(1e-30)
        assert np.max(rel[np.abs(x[r]) > scale[r] * 2.0 ** -6]) <= 2.0 ** -4 + 1e-6        # 3 mantissa bits


def test_fp8_mode_changes_only_the_projection_inputs():
    """With fp8 on, every projection sees de-quantised e4m3 rows of its bf16 input and nothing else changes: a
    layer computed by hand from the pieces equals layer_step, and the distance to the exact run is the
    quantisation noise (a few per cent), not zero and not large."""
    shape = MINI.with_fp8()
    W = mini_weights(seed=33)
    synth.quantize_projections_e4m3(W)
    Wn = weights_to_np(W)
    ids = to_np(synth.make_prompt(shape.vocab, 21, seed=33))
    a = O.prefill(shape, Wn, ids, ((1, 5000),))
    b = O.prefill(MINI, Wn, ids, ((1, 5000),))
    d = rel_err(a.hidden_out[0], b.hidden_out[0])
    assert 1e-4 < d < 0.2
    lw = Wn["layers"][0]
    x = O.f64(Wn["tok_embed"])[ids]
    pos = np.arange(21)

    def lin(v, w):
        c, s = O.quant_rows_e4m3(O._bf16_round(v))
        return (O.f64(c) * O.f64(s)[:, None]) @ O.f64(w).T
    h = O.rmsnorm(x, lw["g_attn"], shape.rms_eps)
    qkv = lin(h, lw["w_qkv"])
    dm = shape.d_model
    q = O.rope(qkv[:, :dm].reshape(21, 4, 16), pos, shape.rope_theta)
    k = O.rope(qkv[:, dm:2 * dm].reshape(21, 4, 16), pos, shape.rope_theta)
    v = qkv[:, 2 * dm:].reshape(21, 4, 16)
    o, _ = O.attend(q, k, v, pos, pos, -1)
    y = x + lin(o, lw["w_o"])
    assert np.allclose(y, a.hidden_after_attn[0], rtol=0, atol=1e-12)
