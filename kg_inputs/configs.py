"""The workload shapes (LLaMA-style decoders of the sizes the paper evaluates, Section 4.1,
plus a tiny one) and the recipe that turns a shape + seed into weights and a prompt.

No arithmetic of the decode method lives here: only shapes, scales and stream ids.
"""
from __future__ import annotations

from dataclasses import dataclass, replace, asdict

import numpy as np

from . import synth
from .synth import TensorId, layer_tid


@dataclass(frozen=True)
class KgShape:
    name: str
    n_layers: int          # L
    d_model: int           # d
    n_heads: int           # H
    head_dim: int          # hd
    d_ffn: int             # F
    vocab: int             # V
    exit_layer: int        # l  (1 <= l < L)
    dtype: str             # "f32" | "bf16": storage type of weights and KV cache
    rms_eps: float = 1e-6
    rope_theta: float = 10000.0
    logit_scale: float = 1.0
    max_seq: int = 256
    page_size: int = 16
    gamma_max: int = 6
    seed: int = 0
    init_std: float = 0.02
    embed_std: float = 0.02
    deep_resid_scale: float = 0.1
    adapter_resid_scale: float = 0.1
    gain_std: float = 0.0  # norm gains are 1 + gain_std * N(0,1); 0 in every benchmark shape
    # workload
    n_prompt: int = 32
    n_gen: int = 64
    eta: float = 0.6
    gamma: int = 6

    def with_(self, **kw) -> "KgShape":
        return replace(self, **kw)

    def as_dict(self):
        return asdict(self)


# Scales marked "calibrated" were chosen once with the oracle (tiny) / the measured accept
# rate (large shapes) so that the top-1 probability spans roughly 0.1..0.99 and the mean
# per-draft accept rate falls in 0.5..0.7; they are frozen here.
CONFIGS = {
    "tiny": KgShape("tiny", 4, 256, 4, 64, 688, 1024, 1, "f32",
                    logit_scale=16.0, max_seq=256, page_size=16, gamma_max=10,
                    deep_resid_scale=0.1, adapter_resid_scale=0.1,
                    n_prompt=32, n_gen=64, eta=0.6, gamma=6),
    "7b": KgShape("7b", 32, 4096, 32, 128, 11008, 32000, 2, "bf16",
                  logit_scale=8.0, max_seq=1024, page_size=16, gamma_max=10,
                  deep_resid_scale=0.03, adapter_resid_scale=0.03,      # measured: accept rate 0.65, CR 2.55, top-1 p 0.23..1.0
                  n_prompt=512, n_gen=256, eta=0.6, gamma=6),
    "13b": KgShape("13b", 40, 5120, 40, 128, 13824, 32000, 2, "bf16",
                   logit_scale=8.0, max_seq=2048 + 512 + 64, page_size=16, gamma_max=10,
                   deep_resid_scale=0.03, adapter_resid_scale=0.03,
                   n_prompt=2048, n_gen=512, eta=0.6, gamma=6),
    "33b": KgShape("33b", 60, 6656, 52, 128, 17920, 32000, 3, "bf16",
                   logit_scale=8.0, max_seq=4096 + 256 + 64, page_size=16, gamma_max=10,
                   deep_resid_scale=0.03, adapter_resid_scale=0.03,
                   n_prompt=4096, n_gen=256, eta=0.6, gamma=8),
}


def get_config(name: str, **overrides) -> KgShape:
    c = CONFIGS[name]
    return c.with_(**overrides) if overrides else c


def param_counts(d: int, F: int, V: int):
    """Closed-form parameter counts of the blocks (norm gains included)."""
    return {
        "adapter": 4 * d * d + 2 * d,            # one attention (q,k,v,o) + two norm gains
        "layer": 4 * d * d + 3 * d * F + 2 * d,  # attention + SwiGLU FFN + two norm gains
        "ffn": 3 * d * F,
        "head": V * d,
    }


# ---- tensor recipe -------------------------------------------------------------------

def tensor_spec(shape: KgShape, name: str, layer: int | None = None):
    """(stream id, (rows, cols), std) of one weight matrix.  `layer` in [0, L) for decoder
    layers, layer == L for the adapter (which has only wqkv and wo)."""
    d, F, V, L = shape.d_model, shape.d_ffn, shape.vocab, shape.n_layers
    f32 = lambda v: float(np.float32(v))      # the C ABI carries these as fp32; products are formed in double
    s = f32(shape.init_std)
    if name == "embed":
        return int(TensorId.EMBED), (V, d), f32(shape.embed_std)
    if name == "head":
        return int(TensorId.HEAD), (V, d), s
    assert layer is not None
    is_adapter = layer == L
    deep = (not is_adapter) and layer >= shape.exit_layer
    out_scale = f32(shape.adapter_resid_scale) if is_adapter else (f32(shape.deep_resid_scale) if deep else 1.0)
    if name == "wqkv":
        return layer_tid(layer, TensorId.WQKV), (3 * d, d), s
    if name == "wo":
        return layer_tid(layer, TensorId.WO), (d, d), s * out_scale
    assert not is_adapter, name
    if name == "wgate":
        return layer_tid(layer, TensorId.WGATE), (F, d), s
    if name == "wup":
        return layer_tid(layer, TensorId.WUP), (F, d), s
    if name == "wdown":
        return layer_tid(layer, TensorId.WDOWN), (d, F), s * out_scale
    raise KeyError(name)


def weight_tensor(shape: KgShape, name: str, layer: int | None = None, force_numpy=False) -> np.ndarray:
    tid, (r, c), std = tensor_spec(shape, name, layer)
    flat = synth.fill_f32(shape.seed, tid, r * c, std, shape.dtype == "bf16", force_numpy=force_numpy)
    return flat.reshape(r, c)


def gain_vector(shape: KgShape, tid: int) -> np.ndarray:
    """Norm gain 1 + gain_std * g (fp32, never rounded to bf16); exactly 1 when gain_std == 0."""
    d = shape.d_model
    g = synth.gauss_ints(shape.seed, tid, 0, d).astype(np.float32) * synth.scale_f32(float(np.float32(shape.gain_std)))
    return (np.float32(1.0) + g).astype(np.float32)


def make_weights(shape: KgShape, force_numpy=False) -> dict:
    """All weights as fp32 numpy arrays (bf16 shapes: every value bf16-representable).
    Layout: every matrix is [out_features, in_features]."""
    d, L = shape.d_model, shape.n_layers
    w = {
        "embed": weight_tensor(shape, "embed", force_numpy=force_numpy),
        "head": weight_tensor(shape, "head", force_numpy=force_numpy),
        "g_final": gain_vector(shape, int(TensorId.GFINAL)),
        "layers": [],
    }
    for i in range(L):
        w["layers"].append({
            "g1": gain_vector(shape, layer_tid(i, TensorId.G1)),
            "g2": gain_vector(shape, layer_tid(i, TensorId.G2)),
            **{n: weight_tensor(shape, n, i, force_numpy) for n in ("wqkv", "wo", "wgate", "wup", "wdown")},
        })
    w["adapter"] = {
        "g_in": gain_vector(shape, layer_tid(L, TensorId.G1)),
        "g_last": gain_vector(shape, layer_tid(L, TensorId.G2)),
        "wqkv": weight_tensor(shape, "wqkv", L, force_numpy),
        "wo": weight_tensor(shape, "wo", L, force_numpy),
    }
    return w


def make_prompt(shape: KgShape, n: int | None = None) -> np.ndarray:
    n = shape.n_prompt if n is None else n
    return synth.uniform_tokens(shape.seed, int(TensorId.PROMPT), n, shape.vocab)


def microbench_state(shape: KgShape, T: int, n_d: int, seed: int) -> dict:
    """Inputs of the verify-step / draft-step microbenchmark: every KV cache holds seeded N(0,1)
    entries for positions [0, T) (rounded to the storage type), the early-feature slots hold
    N(0,1) rows (slot 0 = position T-1, slot 1+j = f_j), plus x_0 and n_d draft token ids.
    Element (pos, head, e) of a cache is element (pos*H + head)*hd + e of its stream."""
    H, hd, d, L = shape.n_heads, shape.head_dim, shape.d_model, shape.n_layers
    bf = shape.dtype == "bf16"
    k, v = [], []
    for i in range(L + 1):
        k.append(synth.fill_f32(seed, layer_tid(i, TensorId.KCACHE), T * H * hd, 1.0, bf).reshape(T, H, hd))
        v.append(synth.fill_f32(seed, layer_tid(i, TensorId.VCACHE), T * H * hd, 1.0, bf).reshape(T, H, hd))
    feat = synth.fill_f32(seed, int(TensorId.HIDDEN), 17 * d, 1.0, False).reshape(17, d)
    toks = synth.uniform_tokens(seed, int(TensorId.DRAFT), 1001, shape.vocab)
    return {"k": k, "v": v, "feat": feat, "x0": int(toks[1000]), "drafts": [int(t) for t in toks[:max(n_d, 0)]]}


# ---- weights regenerated on demand ---------------------------------------------------

class _LazyBlock:
    """One layer's (or the adapter's) tensors, produced when they are read."""

    def __init__(self, owner, layer, names):
        self._owner, self._layer, self._names = owner, layer, names

    def __getitem__(self, name):
        return self._owner._get(self._layer, self._names[name])

    def keys(self):
        return self._names.keys()


class LazyWeights:
    """The same tensors as make_weights, with the same nesting (w["layers"][i]["wqkv"], w["adapter"]["wo"],
    w["head"], ...), produced from their counter streams when they are read and converted to `dtype`.
    For shapes whose weights do not fit in host memory at 8 bytes per value.

    The tensors read first are kept until `budget_bytes` are held; every tensor read after that is
    regenerated on each read into one of two reusable buffers of its shape, so such an array is only valid
    until the second-next read of a tensor of the same shape (a matrix-vector product uses it at once).
    `lazy_weights = True` tells a consumer to take the tensors as they come instead of converting the whole
    collection up front."""
    lazy_weights = True

    def __init__(self, shape: KgShape, dtype=np.float64, budget_bytes: int = 16 << 30):
        self.shape, self.dtype, self.budget = shape, np.dtype(dtype), int(budget_bytes)
        self._held = {}          # (layer, name) -> array kept for good
        self._bytes = 0
        self._scratch = {}       # array shape -> [buffers, next buffer]
        L = shape.n_layers
        mats = ("wqkv", "wo", "wgate", "wup", "wdown")
        self._top = {"embed": (None, "embed"), "head": (None, "head"), "g_final": (None, "g_final")}
        self._layers = [_LazyBlock(self, i, {**{n: n for n in mats}, "g1": "g1", "g2": "g2"}) for i in range(L)]
        self._adapter = _LazyBlock(self, L, {"wqkv": "wqkv", "wo": "wo", "g_in": "g1", "g_last": "g2"})

    def __getitem__(self, key):
        if key == "layers":
            return self._layers
        if key == "adapter":
            return self._adapter
        return self._get(*self._top[key])

    def _make(self, layer, name):
        s = self.shape
        if name == "g_final":
            return gain_vector(s, int(TensorId.GFINAL))
        if name == "g1":
            return gain_vector(s, layer_tid(layer, TensorId.G1))
        if name == "g2":
            return gain_vector(s, layer_tid(layer, TensorId.G2))
        return weight_tensor(s, name, layer)

    def _get(self, layer, name):
        key = (layer, name)
        a = self._held.get(key)
        if a is not None:
            return a
        src = self._make(layer, name)
        nbytes = src.size * self.dtype.itemsize
        if self._bytes + nbytes <= self.budget:
            a = src.astype(self.dtype)
            self._held[key] = a
            self._bytes += nbytes
            return a
        slot = self._scratch.setdefault(src.shape, [[np.empty(src.shape, self.dtype), np.empty(src.shape, self.dtype)], 0])
        a = slot[0][slot[1]]
        slot[1] ^= 1
        np.copyto(a, src)
        return a
