"""The draft / verify / accept controller of the oracle, driven by table-based fake models
(no network): every agreement pattern for small gamma, the discard rule, the 1..gamma+1 yield,
the adapter-cache lag, and the worked example of the paper's Figure 2."""
import itertools

import numpy as np
import pytest

from oracle import kangaroo_oracle as ko


class FakeKangaroo(ko.KangarooOracle):
    """A 'model' whose target and draft are arbitrary functions of the token prefix.

    target(prefix) -> token;  draft(prefix) -> (token, p).  A feature is just the prefix that
    produced it, so the test can check which rows each stage was given."""

    def __init__(self, target, draft, prompt):
        self.target, self.draft = target, draft
        self.P = len(prompt)
        self.tokens = list(prompt)
        self.x0 = target(tuple(prompt))
        self.tokens.append(self.x0)
        self.kv_len = len(prompt)          # shallow == deep cache length
        self.len_A = len(prompt)
        self.f_prev = None
        self.S, self.log, self.gaps = [], [], []
        self.adapter_units = []            # rows handed to the adapter at each call
        self.verify_units = []

    def _shallow_feature(self, tok, pos):
        assert pos == self.kv_len or pos < self.kv_len + 32
        prefix = tuple(self.tokens[: self.P]) + tuple(self._cur_round_tokens(pos)) + (tok,)
        assert len(prefix) == pos + 1
        self._round_toks[pos] = tok
        return prefix

    def _cur_round_tokens(self, pos):
        return [self._round_toks[q] for q in range(self.P, pos)]

    def _draft_head(self, feats, pos0):
        assert pos0 == self.len_A
        self.adapter_units.append(len(feats))
        for i, f in enumerate(feats):
            assert len(f) == pos0 + i + 1          # the feature of position pos0+i
        self.len_A = pos0 + len(feats)
        tok, p = self.draft(feats[-1])
        return tok, p, None

    def _verify_tokens(self, feats, pos0):
        assert pos0 == self.P
        self.verify_units.append(len(feats))
        return [self.target(f) for f in feats], None

    def _adapter_len(self):
        return self.len_A

    def _rollback(self, n_keep):
        self.kv_len = n_keep
        self.len_A = min(self.len_A, n_keep)

    def round(self, *a, **k):
        self._round_toks = {}
        return super().round(*a, **k)


def greedy_reference(target, prompt, n):
    seq = list(prompt)
    out = []
    for _ in range(n):
        t = target(tuple(seq))
        out.append(t)
        seq.append(t)
    return out


def make_target(seed):
    def target(prefix):
        return hash((seed, prefix)) % 50
    return target


@pytest.mark.parametrize("mode", [ko.STOP_KEEP, ko.STOP_DROP])
@pytest.mark.parametrize("gamma", [1, 2, 3, 4])
def test_every_agreement_and_confidence_pattern(gamma, mode):
    """Enumerate, for one round, every pattern of (draft agrees with target?, confidence high?)."""
    target = make_target(1)
    prompt = [3, 1, 4]
    eta = 0.5
    for agree in itertools.product([0, 1], repeat=gamma):
        for conf in itertools.product([0, 1], repeat=gamma):
            def draft(prefix, agree=agree, conf=conf):
                j = len(prefix) - len(prompt) - 1          # draft step index
                t = target(prefix)
                tok = t if agree[j] else (t + 1) % 50
                return tok, (0.9 if conf[j] else 0.2)
            m = FakeKangaroo(target, draft, prompt)
            em = m.round(eta, gamma, mode)
            r = m.log[-1]
            # expected number of drafts
            n_d = 0
            for j in range(gamma):
                if conf[j]:
                    n_d += 1
                else:
                    n_d += 1 if mode == ko.STOP_KEEP else 0
                    break
            assert r["n_drafted"] == n_d
            assert r["M"] == n_d + 1 == m.verify_units[-1]
            k = 0
            while k < n_d and agree[k]:
                k += 1
            assert r["k"] == k
            assert 1 <= len(em) == k + 1 <= gamma + 1                        # 1 .. gamma+1 tokens per target forward
            assert em == greedy_reference(target, prompt + [m.tokens[len(prompt)]], k + 1)   # lossless
            if k < n_d:                                                      # discard after the first reject
                assert em[-1] != r["drafts"][k]
            assert m.kv_len == m.P == len(prompt) + k + 1
            assert m.len_A in (m.P, m.P - 1)
            assert (m.f_prev is not None) == (m.len_A == m.P - 1)
            if m.len_A == m.P - 1:
                assert k == n_d and len(m.f_prev) == m.P                     # the feature at position P-1


@pytest.mark.parametrize("mode", [ko.STOP_KEEP, ko.STOP_DROP])
def test_multi_round_lossless_with_random_tables(mode):
    rng = np.random.default_rng(0)
    for trial in range(30):
        target = make_target(trial)
        agree_p, conf_p = rng.uniform(0.2, 0.95), rng.uniform(0.2, 0.95)
        table = {}

        def draft(prefix):
            if prefix not in table:
                r = np.random.default_rng(hash(prefix) % (2**32))
                t = target(prefix)
                table[prefix] = (t if r.uniform() < agree_p else (t + 7) % 50, float(r.uniform() < conf_p) * 0.7 + 0.2)
            return table[prefix]
        prompt = [1, 2, 3, 4]
        gamma = int(rng.integers(1, 7))
        m = FakeKangaroo(target, draft, prompt)
        out = [m.x0]
        while len(out) < 40:
            out += m.round(0.5, gamma, mode)
        assert out == greedy_reference(target, prompt, len(out))
        assert all(1 <= s <= gamma + 1 for s in m.S)
        assert sum(m.S) == len(out) - 1
        assert all(u in (1, 2) for u in m.adapter_units)


def test_figure2_worked_example():
    """Figure 2: three drafts x'_1..x'_3, drafting stops because conf(x'_3) <= eta, the unit
    [f_0..f_3] (4 rows) is verified, all three drafts are accepted, the next round starts from
    x_4 and its first adapter pass processes the two rows [f_3, f_4]."""
    target = make_target(5)
    prompt = [9, 8, 7]
    confs = {0: 0.9, 1: 0.8, 2: 0.3}

    def draft(prefix):
        j = len(prefix) - len(prompt) - 1
        return target(prefix), confs.get(j % 4, 0.9)
    m = FakeKangaroo(target, draft, prompt)
    em = m.round(0.6, 6, ko.STOP_KEEP)
    r = m.log[-1]
    assert r["n_drafted"] == 3 and r["n_steps"] == 3
    assert m.verify_units == [4]
    assert r["k"] == 3 and len(em) == 4
    assert m.adapter_units == [1, 1, 1]
    assert m.len_A == m.P - 1 and m.f_prev is not None
    m.round(0.6, 6, ko.STOP_KEEP)
    assert m.adapter_units[3] == 2                                           # [f_3, f_4] in one pass
    assert all(u == 1 for u in m.adapter_units[4:])


def test_eta_extremes_with_fakes():
    target = make_target(2)
    prompt = [5, 5]
    draft = lambda prefix: (target(prefix), 0.7)
    for gamma in (1, 3, 6):
        m = FakeKangaroo(target, draft, prompt)
        m.round(0.0, gamma, ko.STOP_KEEP)
        assert m.log[-1]["n_drafted"] == gamma                               # eta = 0: fixed-step drafting (Section 4.2)
        m = FakeKangaroo(target, draft, prompt)
        m.round(1.5, gamma, ko.STOP_DROP)
        assert m.log[-1]["n_drafted"] == 0 and m.verify_units == [1]         # eta > 1 drafts none
        m = FakeKangaroo(target, draft, prompt)
        m.round(1.5, gamma, ko.STOP_KEEP)
        assert m.log[-1]["n_drafted"] == 1                                   # ... or exactly one when the stopped token is kept
    # p == eta stops (Eq. 4 uses <=)
    m = FakeKangaroo(target, lambda prefix: (target(prefix), 0.6), prompt)
    m.round(0.6, 6, ko.STOP_DROP)
    assert m.log[-1]["n_drafted"] == 0
