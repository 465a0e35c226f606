"""CPU oracle for the Kangaroo batch-1 self-speculative decode step.

TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, obviously-correct numpy restatement
of what the paper's method computes.  Only the test-suite, the smoke check and the
benchmark's `cpu_baseline` / `--impl reference` legs may import it; the CUDA product path
never does, and this file imports nothing from the CUDA package.  It shares no code with
the CUDA path: the only common ground is the seeded input generator package `kg_inputs`,
which the *callers* use to build the weights they pass in here.

What is computed (citations are to the paper):

* Target model M^b: a LLaMA-style decoder (Section 4.1: Vicuna); greedy next token
  x_{t+1} = argmax_n M^b_n(. | x^t)  (Section 3, Notation; greedy setting of Definition 1).
* Self-draft model M^s = A o M^b[:l] re-using the target's LM head (Section 3.1, Figure 2);
  the adapter A is one multi-head attention plus two RMS normalisations (Section 3.1,
  Table 2 row "Kangaroo": input norm, attention, last norm; no FFN, no own head).
* Drafting stops when max_n M^s_n(x) <= eta (Eq. 4) or gamma tokens are drafted
  (Section 1: "Given gamma draft tokens ... 1 to gamma+1 new tokens").
* The early features [f_0 .. f_d] are verified by M^b[l:] in one pass (Figure 2); after
  the first draft the target rejects, all later drafts are discarded (Section 3).
* Metrics: compression rate CR (Eq. 1) and consistent token acceptance rate CTAR(w) (Eq. 2).

Precision: `dtype` is the arithmetic type (float64 by default; float32 for the large
shapes where 8 bytes per weight do not fit in host memory).  For "bf16" models there are
exactly two rounding points: the weights handed in are already bf16-representable, and
K / V rows are rounded to bf16 (nearest-even) when written to a cache.

Row independence: every linear map on <= 16 rows is evaluated one row at a time with the
same matrix-vector routine, so a row's result does not depend on how many rows are
processed with it.  Hence oracle-Kangaroo equals oracle-greedy bit for bit.

Pins (tests/test_oracle_*.py): brute-force full-sequence recompute, a torch CPU
composition of one forward, closed forms for RMSNorm / RoPE / softmax confidence, the
paper's parameter counts (Table 2), the controller invariants, the Figure-2 scripted
example, Eq. 1 / Eq. 2 identities.  Unpinned by the paper: the accept-rate range of the
synthetic models (a workload property, recorded not derived).
"""
from __future__ import annotations

import numpy as np

STOP_KEEP = 0   # the token whose confidence is <= eta is kept as a draft (Figure 2 caption)
STOP_DROP = 1   # ... is discarded ("eta > 1 drafts none")


# ----------------------------------------------------------------------------- primitives

def rmsnorm(x, g, eps):
    """RMSNorm(x; g) = g * x / sqrt(mean(x^2) + eps), over the last axis (Section 3.1, [zhang2019root])."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return g * (x / np.sqrt(ms + eps))


def rope(x, pos, theta):
    """Rotary embedding of x[..., H, hd] at integer position `pos`: within a head, element i is
    paired with i + hd/2 and the pair is rotated by the angle pos * theta^(-2i/hd)."""
    hd = x.shape[-1]
    half = hd // 2
    i = np.arange(half, dtype=np.float64)
    ang = (float(pos) * theta ** (-2.0 * i / hd)).astype(x.dtype)
    c, s = np.cos(ang), np.sin(ang)
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def round_bf16(x):
    """Nearest-even rounding to bfloat16 of an array (any float dtype), returned in x's dtype."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    bits = f.view(np.uint32).astype(np.uint64)
    lsb = (bits >> 16) & 1
    r = ((bits + 0x7FFF + lsb) & 0xFFFF0000).astype(np.uint32)
    return r.view(np.float32).astype(x.dtype)


def silu(x):
    return x / (1.0 + np.exp(-x))


def softmax_rows(s):
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=-1, keepdims=True)


def argmax_lowest(z):
    """Index of the maximum; the lowest index wins ties."""
    return int(np.argmax(z))       # numpy returns the first occurrence


def top1_confidence(z):
    """(token, p) with p = softmax(z)[token] = 1 / sum_i exp(z_i - z_max)   (Eq. 4's left side)."""
    tok = argmax_lowest(z)
    p = 1.0 / float(np.sum(np.exp(z - z[tok])))
    return tok, p


def top2_gap(z):
    """Difference between the largest and second largest entry (near-tie diagnostic)."""
    if z.shape[0] < 2:
        return float("inf")
    part = np.partition(z, -2)
    return float(part[-1] - part[-2])


# ----------------------------------------------------------------------------- metrics

def compression_rate(S):
    """Eq. 1: CR = (1/|S|) sum_k s_k."""
    return float(sum(S)) / len(S)


def ctar(S, w):
    """Eq. 2: CTAR(w) = (1/|S|) sum_k I(s_k - w > 0)."""
    return float(sum(1 for s in S if s - w > 0)) / len(S)


# ----------------------------------------------------------------------------- the model

class KVCache:
    """K and V rows of one attention layer for positions [0, length)."""

    def __init__(self, max_seq, H, hd, dtype, storage_bf16):
        self.k = np.zeros((max_seq, H, hd), dtype)
        self.v = np.zeros((max_seq, H, hd), dtype)
        self.length = 0
        self.storage_bf16 = storage_bf16

    def write(self, pos, k, v):
        assert pos == self.length, (pos, self.length)
        if self.storage_bf16:
            k, v = round_bf16(k), round_bf16(v)
        self.k[pos], self.v[pos] = k, v
        self.length = pos + 1

    def truncate(self, n):
        self.length = min(self.length, n)


class KangarooOracle:
    """Target decoder, self-draft model and the draft / verify / accept controller.

    `shape` needs the attributes n_layers, d_model, n_heads, head_dim, d_ffn, vocab,
    exit_layer, dtype ("f32"|"bf16"), rms_eps, rope_theta, logit_scale, max_seq.
    `weights` is the dict built by the input-generator package: matrices are
    [out_features, in_features].
    """

    def __init__(self, shape, weights, dtype=np.float64):
        self.s = shape
        self.dt = np.dtype(dtype)
        self.L, self.l = shape.n_layers, shape.exit_layer
        self.d, self.H, self.hd = shape.d_model, shape.n_heads, shape.head_dim
        assert 1 <= self.l < self.L
        assert self.H * self.hd == self.d
        self.w = self._cast(weights)
        self.reset()

    def _cast(self, w):
        if self.dt == np.float32 or getattr(w, "lazy_weights", False):
            return w                  # a lazy collection hands out tensors of the wanted type one at a time
        if isinstance(w, dict):
            return {k: self._cast(v) for k, v in w.items()}
        if isinstance(w, list):
            return [self._cast(v) for v in w]
        return np.asarray(w, dtype=self.dt)

    # -- state -------------------------------------------------------------------------
    def reset(self):
        s = self.s
        bf = s.dtype == "bf16"
        self.cache = [KVCache(s.max_seq, self.H, self.hd, self.dt, bf) for _ in range(self.L)]
        self.cache_A = KVCache(s.max_seq, self.H, self.hd, self.dt, bf)
        self.P = 0               # position of the round's first token x_0 = number of tokens in the KV caches
        self.x0 = None
        self.f_prev = None       # early feature at position P-1, kept while the adapter cache lags
        self.tokens = []         # prompt + everything emitted so far (x_0 included)
        self.S = []
        self.log = []            # one dict per round
        self.gaps = []           # (kind, position, top-2 gap) of every argmax taken

    # -- linear algebra ----------------------------------------------------------------
    def linear(self, x, W):
        """x[M, in] -> [M, out] = x W^T; one matrix-vector product per row when M <= 16."""
        x = np.atleast_2d(x)
        if x.shape[0] <= 16:
            return np.stack([W @ x[i] for i in range(x.shape[0])])
        return x @ W.T

    # -- blocks ------------------------------------------------------------------------
    def attention_core(self, qkv, pos0, cache):
        """Causal multi-head attention given the raw rows qkv[M, 3d] = [q | k | v] at positions pos0..:
        rotate q and k, append k and v to `cache`, row i attends to keys 0 .. pos0+i.
        Returns concat_heads softmax(q K^T / sqrt(hd)) V, shape [M, d]."""
        M = qkv.shape[0]
        d, H, hd = self.d, self.H, self.hd
        out = np.zeros((M, d), self.dt)
        for i in range(M):
            pos = pos0 + i
            q = rope(qkv[i, 0:d].reshape(H, hd), pos, self.s.rope_theta)
            k = rope(qkv[i, d:2 * d].reshape(H, hd), pos, self.s.rope_theta)
            v = qkv[i, 2 * d:3 * d].reshape(H, hd)
            cache.write(pos, k, v)
            K = cache.k[:pos + 1]                     # [T, H, hd]
            V = cache.v[:pos + 1]
            scores = np.einsum("hd,thd->ht", q, K) / np.sqrt(self.dt.type(hd))
            p = softmax_rows(scores)
            out[i] = np.einsum("ht,thd->hd", p, V).reshape(d)
        return out

    def attention(self, n, pos0, wqkv, wo, cache):
        """Wo . Attn(n) for the normalised rows n[M, d] at positions pos0.., appending their K/V to `cache`."""
        return self.linear(self.attention_core(self.linear(n, wqkv), pos0, cache), wo)

    def decoder_layer(self, h, pos0, i):
        """One LLaMA block: h += Wo Attn(RMSNorm(h)); h += Wdown(SiLU(Wgate n) * (Wup n))."""
        lw = self.w["layers"][i]
        eps = self.s.rms_eps
        h = h + self.attention(rmsnorm(h, lw["g1"], eps), pos0, lw["wqkv"], lw["wo"], self.cache[i])
        n = rmsnorm(h, lw["g2"], eps)
        act = silu(self.linear(n, lw["wgate"])) * self.linear(n, lw["wup"])
        return h + self.linear(act, lw["wdown"])

    def embed(self, toks):
        return np.asarray(self.w["embed"][np.asarray(toks, dtype=np.int64)], dtype=self.dt)

    def shallow(self, toks, pos0):
        """Early features f = M^b[:l](tokens) (Figure 2); appends the shallow layers' KV."""
        h = self.embed(np.atleast_1d(toks))
        for i in range(self.l):
            h = self.decoder_layer(h, pos0, i)
        return h

    def deep(self, f, pos0):
        """M^b[l:] on the rows f (Figure 2: "the remaining layers"); appends the deep layers' KV."""
        h = f
        for i in range(self.l, self.L):
            h = self.decoder_layer(h, pos0, i)
        return h

    def adapter(self, f, pos0):
        """A(f) = RMSNorm_last( f + W^A_o Attn(RMSNorm_in(f)) ) with its own KV cache (Section 3.1, Table 2)."""
        aw = self.w["adapter"]
        eps = self.s.rms_eps
        a = f + self.attention(rmsnorm(f, aw["g_in"], eps), pos0, aw["wqkv"], aw["wo"], self.cache_A)
        return rmsnorm(a, aw["g_last"], eps)

    def head_logits(self, y):
        """Scaled logits z = s * W_head y of rows y[M, d] (the shared LM head, Figure 2)."""
        return self.linear(y, self.w["head"]) * self.dt.type(self.s.logit_scale)

    def target_logits(self, h):
        return self.head_logits(rmsnorm(h, self.w["g_final"], self.s.rms_eps))

    # -- prefill -----------------------------------------------------------------------
    def prefill(self, prompt):
        """All L layers over the prompt, the adapter's K/V for every prompt position, and
        x_0 = argmax M^b(. | prompt)."""
        assert self.P == 0
        prompt = [int(t) for t in prompt]
        n = len(prompt)
        f = self.shallow(prompt, 0)
        self.adapter(f, 0)                                    # fills the adapter KV; output unused
        h = self.deep(f, 0)
        z = self.target_logits(h[n - 1:n])[0]
        self.x0 = argmax_lowest(z)
        self.gaps.append(("prefill", n - 1, top2_gap(z)))
        self.P = n
        self.f_prev = None
        self.tokens = prompt + [self.x0]
        self.last_logits = z
        return self.x0

    # -- plain greedy decoding (the definition the method must reproduce) ---------------
    def ar_step(self):
        """One plain autoregressive step: x_0 through all L layers, next token by argmax."""
        f = self.shallow([self.x0], self.P)
        h = self.deep(f, self.P)
        z = self.target_logits(h)[0]
        tok = argmax_lowest(z)
        self.gaps.append(("ar", self.P, top2_gap(z)))
        self.P += 1
        self.x0 = tok
        self.tokens.append(tok)
        self.last_logits = z
        return tok

    def generate_ar(self, prompt, n_new):
        """x_0 plus n_new-1 further greedy tokens: returns exactly n_new tokens."""
        self.reset()
        out = [self.prefill(prompt)]
        while len(out) < n_new:
            out.append(self.ar_step())
        return out

    # -- hooks the controller calls (overridden by table-driven fakes in the tests) ------
    def _shallow_feature(self, tok, pos):
        return self.shallow([tok], pos)[0]

    def _draft_head(self, feats, pos0):
        """Adapter on the rows `feats` (positions pos0..), LM head on the last row -> (token, p, logits)."""
        y = self.adapter(np.stack(feats), pos0)
        z = self.head_logits(y[-1:])[0]
        tok, p = top1_confidence(z)
        self.gaps.append(("draft", pos0 + len(feats) - 1, top2_gap(z)))
        return tok, p, z

    def _verify_tokens(self, feats, pos0):
        """Target's greedy tokens t_0..t_d for the unit [f_0..f_d] (Figure 2) -> (list, logits[M, V])."""
        h = self.deep(np.stack(feats), pos0)
        z = self.target_logits(h)
        for i in range(z.shape[0]):
            self.gaps.append(("verify", pos0 + i, top2_gap(z[i])))
        return [argmax_lowest(z[i]) for i in range(z.shape[0])], z

    def _adapter_len(self):
        return self.cache_A.length

    def _rollback(self, n_keep):
        """Keep positions [0, n_keep) in the shallow and deep caches; the adapter cache keeps
        min(its length, n_keep)."""
        for c in self.cache:
            c.truncate(n_keep)
        self.cache_A.truncate(n_keep)

    # -- one Kangaroo round ---------------------------------------------------------------
    def round(self, eta, gamma, stop_mode=STOP_KEEP):
        """Draft up to gamma tokens with early exit (Eq. 4), verify the unit in one pass,
        accept the longest matching prefix, discard the rest (Section 3; Figure 2).

        Returns the list of emitted tokens (k accepted drafts followed by the target's token t_k)."""
        P = self.P
        f = []                      # early features f_0 .. f_{n_d}
        xd = []                     # drafts x'_1 .. x'_{n_d}
        conf = []                   # every confidence computed this round
        draft_logits = []
        n_steps = 0
        cur = self.x0
        while True:
            f.append(self._shallow_feature(cur, P + len(xd)))          # f[n_d]
            if len(xd) == gamma:
                break
            PA = self._adapter_len()                                   # adapter cache covers [0, PA)
            rows = f[PA - P:] if PA >= P else [self.f_prev] + f        # catch-up unit [f_prev, f_0] when it lags
            assert len(rows) in (1, 2), (PA, P, len(f))
            tok, p, z = self._draft_head(rows, PA)
            n_steps += 1
            conf.append(p)
            draft_logits.append(z)
            if stop_mode == STOP_DROP and p <= eta:
                break
            xd.append(tok)
            cur = tok
            if stop_mode == STOP_KEEP and p <= eta:
                f.append(self._shallow_feature(cur, P + len(xd)))      # "the stopped token's next early feature"
                break
        n_d = len(xd)
        assert len(f) == n_d + 1
        t, vz = self._verify_tokens(f, P)
        k = 0
        while k < n_d and xd[k] == t[k]:                               # x'_{i} must equal t_{i-1}
            k += 1
        emitted = xd[:k] + [t[k]]
        # rollback: positions P .. P+k hold valid rows; everything after is discarded
        len_A_before = self._adapter_len()
        self._rollback(P + k + 1)
        self.f_prev = f[k] if self._adapter_len() < P + k + 1 else None
        if self.f_prev is not None:
            assert k == n_d and self._adapter_len() == P + k, (k, n_d, self._adapter_len(), P)
        self.P = P + k + 1
        self.x0 = t[k]
        self.tokens.extend(emitted)
        self.S.append(k + 1)
        self.log.append(dict(P=P, n_drafted=n_d, n_steps=n_steps, drafts=list(xd), conf=list(conf),
                             target=list(t), k=k, emitted=list(emitted), M=n_d + 1,
                             adapter_len_before=len_A_before, adapter_len_after=self._adapter_len(),
                             draft_logits=draft_logits, verify_logits=vz))
        return emitted

    def generate(self, prompt, n_new, eta, gamma, stop_mode=STOP_KEEP):
        """x_0 from prefill, then rounds until n_new tokens exist; the last round is truncated so
        that exactly n_new tokens are returned and sum(S) counts only returned tokens (Section 3)."""
        self.reset()
        out = [self.prefill(prompt)]
        while len(out) < n_new:
            em = self.round(eta, gamma, stop_mode)
            room = n_new - len(out)
            if len(em) > room:
                em = em[:room]
                self.S[-1] = room
            out.extend(em)
        return out

    # -- brute force: no cache, whole sequence at once -------------------------------------
    def full_recompute_logits(self, tokens):
        """Target logits for every position of `tokens`, recomputed from scratch with a masked
        [T, T] attention and no cache of any kind (used to pin the cached path)."""
        s = self.s
        T = len(tokens)
        d, H, hd = self.d, self.H, self.hd
        bf = s.dtype == "bf16"
        h = self.embed(tokens)
        mask = np.triu(np.ones((T, T), bool), 1)
        for i in range(self.L):
            lw = self.w["layers"][i]
            n = rmsnorm(h, lw["g1"], s.rms_eps)
            qkv = n @ lw["wqkv"].T
            q = np.stack([rope(qkv[t, 0:d].reshape(H, hd), t, s.rope_theta) for t in range(T)])
            k = np.stack([rope(qkv[t, d:2 * d].reshape(H, hd), t, s.rope_theta) for t in range(T)])
            v = qkv[:, 2 * d:].reshape(T, H, hd)
            if bf:
                k, v = round_bf16(k), round_bf16(v)
            sc = np.einsum("qhd,khd->hqk", q, k) / np.sqrt(self.dt.type(hd))
            sc = np.where(mask[None], -np.inf, sc)
            p = softmax_rows(sc)
            o = np.einsum("hqk,khd->qhd", p, v).reshape(T, d)
            h = h + o @ lw["wo"].T
            n = rmsnorm(h, lw["g2"], s.rms_eps)
            h = h + (silu(n @ lw["wgate"].T) * (n @ lw["wup"].T)) @ lw["wdown"].T
        return (rmsnorm(h, self.w["g_final"], s.rms_eps) @ self.w["head"].T) * self.dt.type(s.logit_scale)
