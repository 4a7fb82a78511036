"""Pins for the oracle's accept rules, prefix sums, samplers and draft: hand-built cases stated in
probabilities, invariants from the paper's text and proofs, and exhaustive enumeration at vocab 8."""
import itertools
import math

import numpy as np
import pytest

import mtad_synth as S
from oracle import mtad_oracle as O

V, GAMMA = 8, 3


def _tables(seed, closeness):
    """Two explicit 'models': conditional tables p(.|context), q(.|context) for every context of length 0..3."""
    rng = np.random.default_rng(seed)
    p, q = {}, {}
    for k in range(GAMMA + 1):
        for ctx in itertools.product(range(V), repeat=k):
            z = rng.standard_normal(V) * 1.5
            p[ctx] = np.exp(O.log_softmax(z[None])[0])
            q[ctx] = np.exp(O.log_softmax((z + closeness * rng.standard_normal(V))[None])[0])
    return p, q


def _chain_inputs(p, q, x):
    logits = np.stack([np.log(p[tuple(x[:i])]) for i in range(len(x) + 1)])
    logq = np.cumsum([math.log(q[tuple(x[:i])][x[i]]) for i in range(len(x))])
    return logits, logq


def test_prefix_sums_are_products_of_probabilities():
    rng = np.random.default_rng(0)
    tr = S.beam_tree(4, 8, 2, 1000, stream=1)
    prob = rng.uniform(0.05, 0.9, size=len(tr.tok))
    LP = O.path_prefix_sums(np.log(prob), tr.parent)
    for n in range(len(tr.tok)):
        prod, m = 1.0, n
        while m >= 0:
            prod *= prob[m]; m = tr.parent[m]
        assert abs(math.exp(LP[n]) - prod) < 1e-15


def test_node_logprobs_pick_the_parent_row():
    rng = np.random.default_rng(1)
    logits = rng.standard_normal((4, 6))
    P = np.exp(logits) / np.exp(logits).sum(-1, keepdims=True)
    tok, parent = [2, 5, 0], [-1, -1, 1]
    lp, lse = O.node_logprobs(logits, tok, parent)
    assert np.allclose(np.exp(lp), [P[0, 2], P[0, 5], P[2, 0]])
    assert np.allclose(lse, np.log(np.exp(logits).sum(-1)))


def _chain_from_probs(p_tok, q_tok, tau):
    LP = np.cumsum(np.log(p_tok)); LQ = np.cumsum(np.log(q_tok))
    return O.accept_chain(LP, LQ, math.log(tau) if tau > 0 else O.NEG_INF)[0]


def test_chain_rule_hand_cases():
    # all prefixes pass: p >= q everywhere
    assert _chain_from_probs([.5, .5, .5], [.4, .4, .4], 0.5) == 3
    # none pass: joint ratios .1, .01, .001
    assert _chain_from_probs([.05, .05, .05], [.5, .5, .5], 0.3) == 0
    # non-monotone: ratio after 1 token 0.2 (fails tau=.5), after 2 tokens 0.2*4=0.8 (passes), after 3: 0.08
    assert _chain_from_probs([.1, .8, .05], [.5, .2, .5], 0.5) == 2
    # a later pass overrides an earlier pass too: ratios .9, .09, .9
    assert _chain_from_probs([.45, .05, .5], [.5, .5, .05], 0.5) == 3
    # strict comparison at equality (ratio exactly tau): p/q = 0.5 -> not accepted
    assert _chain_from_probs([.25], [.5], 0.5) == 0
    # tau = 0 accepts everything with p > 0
    assert _chain_from_probs([1e-30, 1e-30], [.9, .9], 0.0) == 2
    # min(1, p/q) never blocks: ratio 50 passes for tau just below 1
    assert _chain_from_probs([.5], [.01], 0.999) == 1


def test_chain_invariants_on_random_inputs():
    rng = np.random.default_rng(2)
    for _ in range(500):
        g = int(rng.integers(1, 9))
        pt, qt = rng.uniform(.01, 1, g), rng.uniform(.01, 1, g)
        tau = float(rng.uniform(.05, .95))
        eta = _chain_from_probs(pt, qt, tau)
        P, Q = np.cumprod(pt), np.cumprod(qt)
        if eta > 0:
            assert P[eta - 1] / Q[eta - 1] > tau                          # accepted prefix clears the threshold
            if Q[eta - 1] > P[eta - 1]:
                assert (Q[eta - 1] - P[eta - 1]) / P[eta - 1] < 1 / tau - 1  # bounded relative error (Sec. 3.2)
        for j in range(eta, g):
            assert not (min(1.0, P[j] / Q[j]) > tau)                      # every longer prefix fails


def test_gamma_zero_is_plain_autoregressive_sampling():
    rng = np.random.default_rng(3)
    logits = rng.standard_normal((1, 50))
    u = rng.uniform(size=50)
    res = O.verify_from_logits(logits, [], [], [], math.log(0.3), u, chain=True)
    t, _ = O.gumbel_argmax(logits[0], u)
    assert res.eta == 0 and res.out_tok == [t]
    assert abs(res.out_lp[0] - O.log_softmax(logits)[0, t]) < 1e-12


def test_theorem_short_prefixes_always_accepted():
    # proof of the bound gamma_bar >= |log tau| / U: a prefix of length j <= |log tau| / U always passes
    p, q = _tables(7, 0.15)
    U = max(np.max(np.abs(np.log(p[c]) - np.log(q[c]))) for c in p if len(c) < GAMMA)
    for tau in (0.05, 0.2, 0.5):
        jmax = int(math.floor(abs(math.log(tau)) / U))
        assert jmax >= 1 or tau == 0.5
        for x in itertools.product(range(V), repeat=GAMMA):
            logits, logq = _chain_inputs(p, q, x)
            lp, _ = O.node_logprobs(logits, x, list(range(-1, GAMMA - 1)))
            LP = O.path_prefix_sums(lp, list(range(-1, GAMMA - 1)))
            assert np.allclose(np.exp(LP), np.cumprod([p[tuple(x[:i])][x[i]] for i in range(GAMMA)]))
            eta, _ = O.accept_chain(LP, logq, math.log(tau))
            # strictness: the theorem's bound is non-strict, equality has measure zero with these tables
            assert eta >= min(jmax, GAMMA)


def _chi_square_ok(counts, expected, n, min_expected=5.0, z=5.0):
    """Pearson statistic over cells with enough mass (rest pooled); passes if within z sigma of its mean."""
    stat, dof, pool_c, pool_e = 0.0, 0, 0.0, 0.0
    for key, e in expected.items():
        c = counts.get(key, 0)
        if e * n >= min_expected:
            stat += (c - e * n) ** 2 / (e * n); dof += 1
        else:
            pool_c += c; pool_e += e * n
    if pool_e >= min_expected:
        stat += (pool_c - pool_e) ** 2 / pool_e; dof += 1
    dof -= 1
    assert set(counts) <= set(expected)
    return stat < dof + z * math.sqrt(2 * dof), (stat, dof)


@pytest.mark.parametrize("sampler", ["gumbel", "inverse_cdf"])
def test_exact_output_distribution_by_enumeration(sampler):
    """Draft x ~ q (beam sampling of width 1 is ancestral sampling), verify with the chain rule, bonus ~ p.
    The law of the returned block [x_1..x_eta, t] is sum_x q(x) 1[eta(x)] p(t | x_{1:eta}); enumerate it."""
    p, q = _tables(11, 1.5)
    tau = 0.6
    exact = {}
    for x in itertools.product(range(V), repeat=GAMMA):
        qx = math.prod(q[tuple(x[:i])][x[i]] for i in range(GAMMA))
        logits, logq = _chain_inputs(p, q, x)
        LP = np.cumsum([math.log(p[tuple(x[:i])][x[i]]) for i in range(GAMMA)])
        eta = max([j + 1 for j in range(GAMMA) if math.exp(LP[j] - logq[j]) > tau], default=0)
        for t in range(V):
            key = tuple(x[:eta]) + (t,)
            exact[key] = exact.get(key, 0.0) + qx * p[tuple(x[:eta])][t]
    assert abs(sum(exact.values()) - 1.0) < 1e-12
    etas = {len(k) - 1 for k, v in exact.items() if v > 0}
    assert etas == {0, 1, 2, 3}                                   # every accepted length occurs
    rng = np.random.default_rng(5)
    n, counts = 40000, {}
    for _ in range(n):
        x = []
        for i in range(GAMMA):                                    # the oracle's own draft sampler, width 1
            x.append(O.gumbel_top_b(np.log(q[tuple(x)])[None], rng.uniform(size=(1, V)), 1)[0])
        logits, logq = _chain_inputs(p, q, x)
        if sampler == "gumbel":
            res = O.verify_from_logits(logits, x, list(range(-1, GAMMA - 1)), logq, math.log(tau),
                                       rng.uniform(size=V), chain=True)
            key = tuple(res.out_tok)
            assert key[:-1] == tuple(x[:res.eta])
        else:
            lp, _ = O.node_logprobs(logits, x, list(range(-1, GAMMA - 1)))
            eta, _ = O.accept_chain(O.path_prefix_sums(lp, list(range(-1, GAMMA - 1))), logq, math.log(tau))
            key = tuple(x[:eta]) + (O.inverse_cdf_sample(p[tuple(x[:eta])], rng.uniform()),)
        counts[key] = counts.get(key, 0) + 1
    ok, info = _chi_square_ok(counts, exact, n)
    assert ok, info


def test_samplers_at_vocab_8():
    rng = np.random.default_rng(6)
    z = rng.standard_normal(V) * 1.3
    pz = np.exp(O.log_softmax(z[None])[0])
    n = 60000
    counts = np.zeros(V)
    for _ in range(n):
        counts[O.gumbel_argmax(z, rng.uniform(size=V))[0]] += 1
    assert np.all(np.abs(counts / n - pz) < 5 * np.sqrt(pz * (1 - pz) / n))
    # inverse CDF: token k owns an interval of length p_k
    edges = np.concatenate([[0.0], np.cumsum(pz)])
    for k in range(V):
        mid = 0.5 * (edges[k] + edges[k + 1])
        assert O.inverse_cdf_sample(pz, mid) == k
        assert abs((edges[k + 1] - edges[k]) - pz[k]) < 1e-15
    # ties -> lowest index; margin is the gap to the runner-up
    t, gap = O.gumbel_argmax(np.array([1.0, 3.0, 3.0]), np.array([.5, .5, .5]))
    assert t == 1 and gap == 0.0


def test_gumbel_top_b_inclusion_probabilities():
    # ordered pair (i, j) without replacement has probability p_i * p_j / (1 - p_i)
    rng = np.random.default_rng(8)
    s = rng.standard_normal((2, 4))                              # two beams x four tokens, flat index = beam*4+tok
    w = np.exp(s).ravel(); w /= w.sum()
    n, counts = 60000, {}
    for _ in range(n):
        pick = tuple(O.gumbel_top_b(s, rng.uniform(size=(2, 4)), 2))
        assert pick[0] != pick[1]
        counts[pick] = counts.get(pick, 0) + 1
    exact = {(i, j): w[i] * w[j] / (1 - w[i]) for i in range(8) for j in range(8) if i != j}
    ok, info = _chi_square_ok(counts, exact, n)
    assert ok, info


def test_tree_rule_hand_cases():
    #      root -> 0 (d1) -> 2 (d2)
    #           -> 1 (d1) -> 3 (d2)
    parent = [-1, -1, 0, 1]
    ref = [math.log(.5), math.log(.25)]
    lt = math.log(.5)
    # deepest passing wins even if a shallower node has a larger ratio
    LP = np.log([.9, .1, .13, .01])
    assert O.accept_tree(LP, parent, ref, lt)[:3] == (2, 2, [0, 2])
    # same depth: higher target likelihood wins
    LP = np.log([.3, .4, .01, .01])
    assert O.accept_tree(LP, parent, ref, lt)[:3] == (1, 1, [1])
    # exact LP tie at the same depth: lowest index
    LP = np.log([.4, .4, .01, .01])
    w, eta, path, _, tie = O.accept_tree(LP, parent, ref, lt)
    assert (w, eta, path, tie) == (0, 1, [0], 0.0)
    # nobody passes -> root, eta 0, empty path
    LP = np.log([.2, .2, .1, .1])
    assert O.accept_tree(LP, parent, ref, lt)[:3] == (-1, 0, [])
    # a child may pass although its parent failed (joint likelihood recovers)
    LP = np.log([.2, .01, .19, .001])
    assert O.accept_tree(LP, parent, ref, lt)[:3] == (2, 2, [0, 2])
    # strict threshold: ratio exactly tau fails
    LP = np.log([.25, .01, .01, .001])
    assert O.accept_tree(LP, parent, ref, lt)[1] == 0


def test_chain_shaped_tree_equals_chain_rule_and_tree_never_shorter():
    rng = np.random.default_rng(9)
    for trial in range(300):
        tr = S.beam_tree(4, 4, 2, 1000, stream=trial)
        lp = -rng.exponential(7.0, size=len(tr.tok))
        LP = O.path_prefix_sums(lp, tr.parent)
        log_tau = math.log(float(rng.uniform(.05, .9)))
        w, eta_tree, path, _, _ = O.accept_tree(LP, tr.parent, tr.logq_ref, log_tau)
        assert [tr.depth[n] for n in path] == list(range(1, eta_tree + 1))
        # the output beam alone, as a chain and as a chain-shaped tree
        LPb = [LP[n] for n in tr.best_path]
        eta_chain, m1 = O.accept_chain(LPb, tr.logq_ref, log_tau)
        wc, eta_ct, pc, m2, _ = O.accept_tree(LPb, list(range(-1, 3)), tr.logq_ref, log_tau)
        assert (eta_ct, pc, m1) == (eta_chain, list(range(eta_chain)), m2)
        assert eta_tree >= eta_chain                                # Sec. 3.3 theorem, per instance
        # sibling order does not matter (no exact ties with continuous values)
        perm = list(range(len(tr.tok)))
        for d in range(1, 5):
            idx = [i for i in perm if tr.depth[i] == d]
            sh = list(rng.permutation(idx))
            for a, b in zip(idx, sh):
                perm[a] = b
        inv = {old: new for new, old in enumerate(perm)}
        parent2 = [(-1 if tr.parent[o] < 0 else inv[tr.parent[o]]) for o in perm]
        if all(p < i for i, p in enumerate(parent2)):
            LP2 = [LP[o] for o in perm]
            w2, eta2, path2, _, _ = O.accept_tree(LP2, parent2, tr.logq_ref, log_tau)
            assert eta2 == eta_tree and [perm[n] for n in path2] == path


def test_draft_beam_bookkeeping():
    """Structure of the beam-sampling draft: b distinct first tokens, node_logq = sum of aux log-probs along the
    path, x** has the largest final joint q, width 1 reduces to ancestral sampling with the same noise."""
    from oracle.adapters import oracle_model
    shape = S.WORKLOADS["tiny"].aux
    model = oracle_model(S.make_model(shape, 1))
    gamma, b, L = 3, 4, 0
    cap = 40
    cache = np.zeros((shape.layers, 2, shape.n_kv_heads, cap, shape.head_dim), dtype=np.uint16)
    pend = S.token_ids(0, 31, 5, shape.vocab).tolist()
    u = S.uniforms(0, 32, gamma * b * shape.vocab).view(gamma, b, shape.vocab).numpy()
    dr = O.draft_beam(model, cache, L, pend, gamma, b, u)
    assert len(dr.tok) == gamma * b and dr.depth == [1] * b + [2] * b + [3] * b
    assert len(set(dr.tok[:b])) == b and all(p == -1 for p in dr.parent[:b])
    pairs = {(dr.parent[n], dr.tok[n]) for n in range(len(dr.tok))}
    assert len(pairs) == len(dr.tok)
    finals = [n for n in range(len(dr.tok)) if dr.depth[n] == gamma]
    assert dr.best_path[-1] in finals and dr.logq[dr.best_path[-1]] == max(dr.logq[n] for n in finals)
    assert dr.logq_ref == [dr.logq[n] for n in dr.best_path]
    # joint log q along x** equals per-token aux log-softmax values from causal token-by-token decoding
    seq = pend + [dr.tok[n] for n in dr.best_path]
    c2 = np.zeros_like(cache)
    acc, want = 0.0, []
    for i, t in enumerate(seq[:-1]):
        lg = O.decoder_rows(model, c2, i, [t], [i], [i], [[i]])
        if i >= len(pend) - 1:
            acc += O.log_softmax(lg)[0, seq[i + 1]]
            want.append(acc)
    assert np.allclose(want, dr.logq_ref, atol=1e-10)
    # width 1: each step is one Gumbel-max draw from q(. | prefix)
    cache1 = np.zeros_like(cache)
    d1 = O.draft_beam(model, cache1, L, pend, gamma, 1, u[:, :1])
    c3 = np.zeros_like(cache)
    for i, t in enumerate(pend[:-1]):
        O.decoder_rows(model, c3, i, [t], [i], [i], [[i]])
    cur, pos = pend[-1], len(pend) - 1
    for step in range(gamma):
        lg = O.decoder_rows(model, c3, pos, [cur], [pos], [pos], [[pos]])[0]
        cur, _ = O.gumbel_argmax(lg, u[step, 0]); pos += 1
        assert cur == d1.tok[step]


def test_aux_commit_equals_rerunning_the_accepted_tokens():
    """After a draft and the roll-forward of the auxiliary cache, the next draft step must see exactly what causal
    decoding of the committed tokens would have produced, whether or not the last drafted layer was accepted."""
    from oracle.adapters import oracle_model
    shape = S.WORKLOADS["tiny"].aux
    model = oracle_model(S.make_model(shape, 1))
    gamma, b, cap = 3, 3, 64
    for accept_len in (0, 2, 3):
        cache = np.zeros((shape.layers, 2, shape.n_kv_heads, cap, shape.head_dim), dtype=np.uint16)
        ctx = S.token_ids(0, 41, 6, shape.vocab).tolist()
        for i, t in enumerate(ctx[:-1]):
            O.decoder_rows(model, cache, i, [t], [i], [i], [[i]])
        L, pend = len(ctx) - 1, [ctx[-1]]
        u = S.uniforms(0, 42 + accept_len, gamma * b * shape.vocab).view(gamma, b, shape.vocab).numpy()
        dr = O.draft_beam(model, cache, L, pend, gamma, b, u)
        accepted = dr.best_path[:accept_len]
        bonus = 77
        L2, pend2 = O.aux_commit(cache, L, pend, dr, accepted, bonus, gamma)
        committed = ctx + [dr.tok[n] for n in accepted] + [bonus]
        assert L2 + len(pend2) == len(committed) and pend2[-1] == bonus
        assert committed[L2:] == pend2
        # next step through the rolled-forward cache vs from scratch
        vis = [[L2 + i for i in range(r + 1)] for r in range(len(pend2))]
        got = O.decoder_rows(model, cache, L2, pend2, [L2 + i for i in range(len(pend2))],
                             [L2 + i for i in range(len(pend2))], vis)[-1]
        c2 = np.zeros_like(cache)
        for i, t in enumerate(committed):
            ref = O.decoder_rows(model, c2, i, [t], [i], [i], [[i]])[0]
        assert np.max(np.abs(ref - got)) < 1e-10


# ----------------------------------------------------------------------------------------------------------------
# warped rows (App. F: top-k, renormalise, then top-p)
# ----------------------------------------------------------------------------------------------------------------

def test_warp_row_hand_computed():
    z = np.log(np.array([0.5, 0.3, 0.15, 0.05]))
    # top-3 -> (0.5, 0.3, 0.15) / 0.95; cumulative 0.526, 0.842 > 0.8 -> two tokens, 5/8 and 3/8
    out, _ = O.warp_row(z, 3, 0.8)
    assert np.allclose(np.exp(out), [5 / 8, 3 / 8, 0, 0], atol=1e-12)
    # top-4 keeps everything; cumulative 0.5, 0.8, 0.95 > 0.9 -> three tokens, 10/19, 6/19, 3/19
    out, margin = O.warp_row(z, 4, 0.9)
    assert np.allclose(np.exp(out), [10 / 19, 6 / 19, 3 / 19, 0], atol=1e-12)
    assert abs(margin - 0.05) < 1e-12
    # k = 1 is greedy decoding (Sec. 2.1)
    out, _ = O.warp_row(np.array([0.1, 2.0, -1.0, 1.9]), 1, 0.9)
    assert np.exp(out).tolist() == [0, 1, 0, 0]
    # the order of the tokens in the row does not matter
    perm = [2, 0, 3, 1]
    out_p, _ = O.warp_row(z[perm], 3, 0.8)
    assert np.allclose(np.exp(out_p), np.array([5 / 8, 3 / 8, 0, 0])[perm], atol=1e-12)


def test_warp_row_without_limits_is_log_softmax():
    rng = np.random.default_rng(5)
    z = rng.normal(size=37)
    out, margin = O.warp_row(z, 37, 1.0)
    assert np.allclose(out, O.log_softmax(z[None])[0], atol=1e-12)
    out, _ = O.warp_row(z, 1000, 1.0)
    assert np.allclose(out, O.log_softmax(z[None])[0], atol=1e-12)


def test_warp_row_is_the_smallest_subset_above_top_p():
    """Brute force over all subsets of a 7-token row: the kept set is a smallest subset of the top-k tokens whose
    renormalised mass is larger than top_p, and the heaviest among those; kept probabilities keep their ratios."""
    import itertools
    rng = np.random.default_rng(11)
    for trial in range(40):
        z = rng.normal(scale=1.5, size=7)
        k = int(rng.integers(2, 8))
        top_p = float(rng.uniform(0.3, 0.97))
        out, margin = O.warp_row(z, k, top_p)
        kept = [i for i in range(7) if np.isfinite(out[i])]
        assert abs(np.exp(out[kept]).sum() - 1) < 1e-12
        topk = sorted(range(7), key=lambda i: -z[i])[:k]
        assert set(kept) <= set(topk)
        p = np.exp(z[topk]) / np.exp(z[topk]).sum()
        mass = dict(zip(topk, p))
        best = None
        for n in range(1, k + 1):
            ok = [s for s in itertools.combinations(topk, n) if sum(mass[i] for i in s) > top_p]
            if ok:
                best = max(ok, key=lambda s: sum(mass[i] for i in s))
                break
        if best is None:
            best = tuple(topk)
        if margin > 1e-9:
            assert set(kept) == set(best)
        ref = kept[0]
        for i in kept:
            assert abs((out[i] - out[ref]) - (z[i] - z[ref])) < 1e-12


def test_warped_verification_drops_tokens_outside_the_kept_set():
    rng = np.random.default_rng(3)
    V, g = 12, 3
    logits = rng.normal(scale=2.0, size=(g + 1, V))
    warped, _ = O.warp_rows(logits, 4, 0.9)
    u = rng.uniform(0.01, 0.99, size=V)
    # a draft whose first token lies outside the first row's kept set can never be accepted, however unlikely q
    dropped = int(np.argmin(logits[0]))
    kept_next = [int(np.argmax(logits[i])) for i in range(1, g)]
    r = O.verify_from_logits(logits, [dropped] + kept_next, list(range(-1, g - 1)), [-50.0] * g, np.log(0.1), u,
                             chain=True, warp=(4, 0.9))
    assert r.eta == 0 and np.isfinite(warped[0, r.out_tok[0]])
    # the most likely token of every row is always kept: that draft passes against a small enough q
    best = [int(np.argmax(logits[i])) for i in range(g)]
    r = O.verify_from_logits(logits, best, list(range(-1, g - 1)), [-50.0] * g, np.log(0.1), u, chain=True,
                             warp=(4, 0.9))
    assert r.eta == g and np.isfinite(warped[g, r.out_tok[-1]])
    # warping that keeps everything changes nothing
    a = O.verify_from_logits(logits, best, list(range(-1, g - 1)), [-3.0, -6.0, -9.0], np.log(0.3), u, chain=True)
    b = O.verify_from_logits(logits, best, list(range(-1, g - 1)), [-3.0, -6.0, -9.0], np.log(0.3), u, chain=True,
                             warp=(V, 1.0))
    assert a.eta == b.eta and a.out_tok == b.out_tok and np.allclose(a.out_lp, b.out_lp, atol=1e-12)


# ----------------------------------------------------------------------------------------------------------------
# vanilla speculative decoding (Sec. 2.2)
# ----------------------------------------------------------------------------------------------------------------

def test_spd_accept_plus_residual_is_the_target_distribution():
    """The identity that makes the rule lossless, from the oracle's own pieces at vocab 8:
    q(y) min(1, p(y)/q(y)) + (1 - sum_x q(x) min(1, p(x)/q(x))) * res(y) / sum(res) = p(y)."""
    p, q = _tables(21, 0.8)
    for ctx in [(), (3,), (1, 6)]:
        lp, lq = np.log(p[ctx]), np.log(q[ctx])
        res = O.spd_residual(lp, lq)
        acc = q[ctx] * np.minimum(1.0, p[ctx] / q[ctx])
        out = acc + (1.0 - acc.sum()) * res / res.sum()
        assert np.allclose(out, p[ctx], atol=1e-12)
        assert np.all(res[p[ctx] <= q[ctx]] == 0) and np.all(res >= 0)


def test_spd_threshold_stop_and_identical_models():
    p, q = _tables(22, 1.0)
    x = [2, 5, 1]
    logits, _ = _chain_inputs(p, q, x)
    logq_rows = np.stack([np.log(q[tuple(x[:i])]) for i in range(len(x))])
    u_res = np.random.default_rng(0).uniform(0.01, 0.99, size=V)
    ratio = [min(1.0, p[tuple(x[:i])][x[i]] / q[tuple(x[:i])][x[i]]) for i in range(3)]
    # every u below its ratio: all accepted, the extra token is a draw from the row after the chain
    r = O.spd_from_logits(logits, x, logq_rows, [0.999 * a for a in ratio], u_res)
    assert r.eta == 3 and r.out_tok[:3] == x
    assert r.out_tok[3] == O.gumbel_argmax(logits[3], u_res)[0]
    # the threshold in u at a position with ratio < 1, and the stop at the first rejection
    k = next(i for i in range(3) if ratio[i] < 1.0)
    u = [0.999 * a for a in ratio]
    u[k] = min(0.999999, ratio[k] * 1.001)
    r = O.spd_from_logits(logits, x, logq_rows, u, u_res)
    assert r.eta == k and len(r.out_tok) == k + 1
    res = O.spd_residual(np.log(p[tuple(x[:k])]), logq_rows[k])
    assert res[r.out_tok[-1]] > 0                                  # resampled where p exceeds q
    with np.errstate(divide="ignore"):
        assert r.out_tok[-1] == O.gumbel_argmax(np.log(res), u_res)[0]
    # identical models: the ratio is 1 everywhere, every draft is accepted whatever u
    lp_rows = np.stack([np.log(p[tuple(x[:i])]) for i in range(len(x))])
    r = O.spd_from_logits(logits, x, lp_rows, [0.999999, 0.5, 1e-9], u_res)
    assert r.eta == 3


def test_spd_first_token_frequencies_follow_the_target():
    """Monte-Carlo over seeded uniforms at vocab 8: the first emitted token (accepted draft or resampled) is
    distributed as the target's first row (chi-square, 7 degrees of freedom)."""
    p, q = _tables(23, 1.2)
    rng = np.random.default_rng(1)
    n = 6000
    logits = np.log(p[()])[None].repeat(2, axis=0)
    counts = np.zeros(V)
    for _ in range(n):
        x0 = int(rng.choice(V, p=q[()]))
        r = O.spd_from_logits(np.stack([np.log(p[()]), np.log(p[(x0,)])]), [x0], np.log(q[()])[None],
                              [float(rng.uniform(1e-12, 1))], rng.uniform(1e-12, 1, size=V))
        counts[r.out_tok[0]] += 1
    chi2 = float(np.sum((counts - n * p[()]) ** 2 / (n * p[()])))
    assert chi2 < 24.3          # 99.9 % quantile of chi-square with 7 degrees of freedom


def test_draft_beam_keep_all_candidates():
    """The wider tree (every layer records b * b candidates) contains the paper's tree: its kept beams are the same
    nodes with the same likelihoods and the same x**; the extra candidates are leaves without a cache row whose
    joint log q is the parent's plus the auxiliary log-probability of their token, and a beam's children come in
    decreasing order of perturbed score."""
    from oracle.adapters import oracle_model
    shape = S.WORKLOADS["tiny"].aux
    model = oracle_model(S.make_model(shape, 1))
    gamma, b, L, cap = 3, 3, 0, 48
    pend = S.token_ids(0, 51, 4, shape.vocab).tolist()
    u = S.uniforms(0, 52, gamma * b * shape.vocab).view(gamma, b, shape.vocab).numpy()
    mk = lambda: np.zeros((shape.layers, 2, shape.n_kv_heads, cap, shape.head_dim), dtype=np.uint16)
    base = O.draft_beam(model, mk(), L, pend, gamma, b, u)
    wide = O.draft_beam(model, mk(), L, pend, gamma, b, u, keep_all=True)
    assert len(wide.tok) == gamma * b * b and wide.depth == sum(([s + 1] * (b * b) for s in range(gamma)), [])
    kept = [n for n in range(len(wide.tok)) if wide.slot[n] >= 0]
    assert len(kept) == gamma * b and sorted(wide.slot[n] for n in kept) == list(range(gamma * b))
    by_slot = {wide.slot[n]: n for n in kept}
    for k in range(gamma * b):                      # beam k of the plain tree == the kept node with slot k
        n = by_slot[k]
        assert wide.tok[n] == base.tok[k] and abs(wide.logq[n] - base.logq[k]) < 1e-12
        assert (wide.parent[n] == -1) == (base.parent[k] == -1)
        if base.parent[k] >= 0:
            assert wide.slot[wide.parent[n]] == base.parent[k]
    assert [wide.slot[n] for n in wide.best_path] == base.best_path and np.allclose(wide.logq_ref, base.logq_ref)
    # leaves: never parents, no cache row; parents are kept nodes of the layer before
    for n in range(len(wide.tok)):
        p = wide.parent[n]
        assert p < n and (p == -1 or (wide.slot[p] >= 0 and wide.depth[p] == wide.depth[n] - 1))
    # children of one beam: distinct tokens, and log q(child) - log q(parent) is the aux log-softmax of the token after
    # the parent's path (causal decoding from scratch)
    n = max(i for i in range(len(wide.tok)) if wide.slot[i] < 0)          # a leaf of the last layer
    path = []
    c = n
    while c >= 0:
        path.append(c); c = wide.parent[c]
    path.reverse()
    seq = pend + [wide.tok[i] for i in path]
    c2 = mk()
    for i, t in enumerate(seq[:-1]):
        lg = O.decoder_rows(model, c2, i, [t], [i], [i], [[i]])
    want = O.log_softmax(lg)[0, seq[-1]]
    parent_lq = wide.logq[wide.parent[n]] if wide.parent[n] >= 0 else 0.0
    assert abs((wide.logq[n] - parent_lq) - want) < 1e-10
    sib = [i for i in range(len(wide.tok)) if wide.parent[i] == wide.parent[n] and wide.depth[i] == wide.depth[n]]
    assert len({wide.tok[i] for i in sib}) == len(sib) == b


def test_aux_commit_with_an_accepted_leaf():
    """A recorded candidate that was not kept as a beam has no row in the auxiliary cache: when the verification
    accepts it (as the last node of the path) it must wait, like a node of the last layer, to be replayed."""
    from oracle.adapters import oracle_model
    shape = S.WORKLOADS["tiny"].aux
    model = oracle_model(S.make_model(shape, 1))
    gamma, b, cap = 3, 2, 64
    cache = np.zeros((shape.layers, 2, shape.n_kv_heads, cap, shape.head_dim), dtype=np.uint16)
    ctx = S.token_ids(0, 61, 5, shape.vocab).tolist()
    for i, t in enumerate(ctx[:-1]):
        O.decoder_rows(model, cache, i, [t], [i], [i], [[i]])
    L, pend = len(ctx) - 1, [ctx[-1]]
    u = S.uniforms(0, 62, gamma * b * shape.vocab).view(gamma, b, shape.vocab).numpy()
    dr = O.draft_beam(model, cache, L, pend, gamma, b, u, keep_all=True)
    leaf = next(n for n in range(len(dr.tok)) if dr.slot[n] < 0 and dr.depth[n] == 2)
    accepted = [dr.parent[leaf], leaf]
    L2, pend2 = O.aux_commit(cache, L, pend, dr, accepted, 9, gamma)
    committed = ctx + [dr.tok[n] for n in accepted] + [9]
    assert committed[L2:] == pend2 and pend2 == [dr.tok[leaf], 9] and L2 == L + 1 + 1
    vis = [[L2 + i for i in range(r + 1)] for r in range(len(pend2))]
    got = O.decoder_rows(model, cache, L2, pend2, [L2 + i for i in range(2)], [L2 + i for i in range(2)], vis)[-1]
    c2 = np.zeros_like(cache)
    for i, t in enumerate(committed):
        want = O.decoder_rows(model, c2, i, [t], [i], [i], [[i]])[0]
    assert np.max(np.abs(got - want)) < 1e-9


# ----------------------------------------------------------------------------------------------------------------
# the margins that decide which device decisions the parity tests compare
# ----------------------------------------------------------------------------------------------------------------

def test_warp_row_margin_hand_computed_and_protective():
    z = np.log(np.array([0.5, 0.3, 0.15, 0.05]))
    # top-3 of (0.5, 0.3, 0.15, 0.05), top_p 0.8: the top-k boundary lies ln 3 apart in logits; the partial sums are
    # 0.5 / 0.95 (0.274 from 0.8) and 0.8 / 0.95 (0.0421 above it): the closest decision is the last one
    _, margin = O.warp_row(z, 3, 0.8)
    assert abs(margin - (0.8 / 0.95 - 0.8)) < 1e-12
    # with top_p out of the way (never reached before the last token) only the top-k boundary is left
    _, margin = O.warp_row(z, 2, 1.0)
    assert abs(margin - min(math.log(0.3 / 0.15), 1.0 - 0.5 / 0.8)) < 1e-12
    # what the margin promises: logits moved by less than a quarter of it keep exactly the same tokens (a partial sum
    # moves by at most e^(2 d) - 1 < margin, the gap across the top-k boundary by at most 2 d < margin)
    rng = np.random.default_rng(11)
    for trial in range(200):
        V = int(rng.integers(4, 12))
        zr = rng.normal(size=V) * 2.0
        k, top_p = int(rng.integers(1, V + 1)), float(rng.uniform(0.3, 0.99))
        out, m = O.warp_row(zr, k, top_p)
        if not np.isfinite(m) or m <= 0:
            continue
        d = rng.uniform(-1, 1, size=V) * min(m, 1.0) / 4.0 * 0.999
        out2, _ = O.warp_row(zr + d, k, top_p)
        assert np.array_equal(np.isfinite(out), np.isfinite(out2)), (trial, m)


def test_spd_robust_margin_is_the_gap_under_the_worst_perturbation():
    rng = np.random.default_rng(5)
    V, g, tol = 9, 3, 2e-3
    seen_reject = seen_accept = 0
    for trial in range(300):
        logits = rng.normal(size=(g + 1, V)) * 2.0
        logq = O.log_softmax(rng.normal(size=(g, V)) * 2.0)
        tok = [int(t) for t in rng.integers(0, V, size=g)]
        u_acc = rng.uniform(0.01, 0.99, size=g)
        u_res = rng.uniform(0.01, 0.99, size=V)
        r = O.spd_from_logits(logits, tok, logq, u_acc, u_res, tol=tol)
        assert r.margin_bonus_robust <= r.margin_bonus + 1e-12
        if r.eta == g:
            # every token accepted: the draw is from the target's next row, log p within +-tol moves the winner's
            # lead by at most 2 tol
            assert abs(r.margin_bonus_robust - (r.margin_bonus - 2 * tol)) < 1e-9
            seen_accept += 1
            continue
        seen_reject += 1
        if r.margin_bonus_robust <= 0:
            continue
        # a positive robust margin promises the same resampled token for any log p within +-tol of the row
        logp = O.log_softmax(logits)
        noise = -np.log(-np.log(u_res))
        for _ in range(20):
            lp2 = logp[r.eta] + rng.uniform(-tol, tol, size=V)
            with np.errstate(divide="ignore"):
                z2 = np.log(np.maximum(0.0, np.exp(lp2) - np.exp(logq[r.eta])))
            assert int(np.argmax(z2 + noise)) == r.out_tok[-1], trial
    assert seen_reject > 50 and seen_accept > 5


def test_draft_beam_on_warped_rows():
    """The draft on warped auxiliary rows (App. F): without limits it is the plain draft; with limits every drafted
    token lies in its row's kept set and its conditional log-likelihood is the warped row's, recomputed by causal
    decoding from scratch; rows that keep fewer pairs than the beam width give layers with fewer nodes."""
    from oracle.adapters import oracle_model
    shape = S.WORKLOADS["tiny"].aux
    model = oracle_model(S.make_model(shape, 1))
    gamma, b, L, cap = 3, 3, 0, 48
    V = shape.vocab
    pend = S.token_ids(0, 61, 3, V).tolist()
    u = S.uniforms(0, 62, gamma * b * V).view(gamma, b, V).numpy()
    mk = lambda: np.zeros((shape.layers, 2, shape.n_kv_heads, cap, shape.head_dim), dtype=np.uint16)
    base = O.draft_beam(model, mk(), L, pend, gamma, b, u)
    same = O.draft_beam(model, mk(), L, pend, gamma, b, u, warp=(V, 1.0))
    assert same.tok == base.tok and same.parent == base.parent and np.allclose(same.logq, base.logq, atol=1e-12)

    def check(dr, top_k, top_p):
        for n in range(len(dr.tok)):
            path = []
            c = n
            while c >= 0:
                path.append(c); c = dr.parent[c]
            path.reverse()
            seq = pend + [dr.tok[i] for i in path]
            c2 = mk()
            for i, t in enumerate(seq[:-1]):
                lg = O.decoder_rows(model, c2, i, [t], [i], [i], [[i]])
            row, _ = O.warp_row(lg[0], top_k, top_p)
            assert np.isfinite(row[seq[-1]]), n                      # never a dropped token
            parent_lq = dr.logq[dr.parent[n]] if dr.parent[n] >= 0 else 0.0
            assert abs((dr.logq[n] - parent_lq) - row[seq[-1]]) < 1e-9, n

    w = O.draft_beam(model, mk(), L, pend, gamma, b, u, warp=(5, 0.9))
    assert np.isfinite(w.margin_warp) and len(w.tok) <= gamma * b and w.depth == sorted(w.depth)
    check(w, 5, 0.9)
    # two kept tokens per row and three beams wanted: layers of 2, 3 (of 2 x 2 pairs), 3 nodes
    w2 = O.draft_beam(model, mk(), L, pend, gamma, b, u, warp=(2, 1.0))
    assert [w2.depth.count(d) for d in (1, 2, 3)] == [2, 3, 3]
    assert sorted(w2.slot[n] for n in range(len(w2.tok))) == [0, 1, 3, 4, 5, 6, 7, 8]
    check(w2, 2, 1.0)
    # greedy rows (one kept token each): a single chain, whatever the beam width
    w1 = O.draft_beam(model, mk(), L, pend, gamma, b, u, warp=(1, 1.0))
    assert w1.parent == [-1, 0, 1] and w1.best_path == [0, 1, 2]
    check(w1, 1, 1.0)
    # every candidate kept, on warped rows: the kept beams are those of the plain warped draft
    wk = O.draft_beam(model, mk(), L, pend, gamma, b, u, keep_all=True, warp=(5, 0.9))
    kept = {wk.slot[n]: n for n in range(len(wk.tok)) if wk.slot[n] >= 0}
    assert [wk.tok[kept[k]] for k in sorted(kept)] == [w.tok[n] for n in sorted(range(len(w.tok)), key=lambda n: w.slot[n])]
    check(wk, 5, 0.9)
