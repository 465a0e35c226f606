"""ctypes binding of include/kangaroo.h: argument marshalling only.

torch is used for the device arena, the stream handle and nothing else.  The library must be
present: there is no fallback path of any kind.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from .build import lib_path

KG_M_MAX = 16
KG_GAMMA_MAX = KG_M_MAX - 1
KG_F32, KG_BF16 = 0, 1
STOP_KEEP, STOP_DROP = 0, 1

KG_OK, KG_E_ARG, KG_E_STATE, KG_E_NOMEM, KG_E_SEQ_FULL, KG_E_CUDA, KG_E_TIMEOUT, KG_E_LIMIT, KG_E_INTERNAL = 0, -1, -2, -3, -4, -5, -6, -7, -8

EXPORTS = [
    "kg_workspace_bytes", "kg_init_model", "kg_free_model", "kg_reset", "kg_prefill", "kg_prefill_device",
    "kg_draft", "kg_verify", "kg_decode", "kg_decode_ar", "kg_generate", "kg_read_tokens", "kg_read_S", "kg_read_round_log",
    "kg_debug_logits", "kg_read_weight", "kg_debug_fill_state", "kg_op_scratch_bytes", "kg_op_linear",
    "kg_op_lm_head", "kg_op_lm_head_noalloc", "kg_op_attention", "kg_strerror",
    "kg_last_cuda_error", "kg_debug_force_simple", "kg_debug_force_simple_ops", "kg_debug_set_wait_budget", "kg_debug_skip_barrier_arrival",
    "kg_debug_set_prefill_mode", "kg_op_gemm",
]


class KgConfig(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32),
        ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
        ("d_ffn", C.c_int32), ("vocab", C.c_int32),
        ("exit_layer", C.c_int32), ("dtype", C.c_int32),
        ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("logit_scale", C.c_float),
        ("max_seq", C.c_int32), ("page_size", C.c_int32), ("gamma_max", C.c_int32),
        ("debug_logits", C.c_int32), ("page_shuffle", C.c_int32),
        ("seed", C.c_uint64),
        ("init_std", C.c_float), ("embed_std", C.c_float), ("deep_resid_scale", C.c_float),
        ("adapter_resid_scale", C.c_float), ("gain_std", C.c_float),
    ]


class KgWeights(C.Structure):
    _fields_ = [
        ("embed_dev", C.c_void_p), ("head_dev", C.c_void_p), ("g_final_dev", C.c_void_p),
        ("wqkv_dev", C.POINTER(C.c_void_p)), ("wo_dev", C.POINTER(C.c_void_p)),
        ("wgate_dev", C.POINTER(C.c_void_p)), ("wup_dev", C.POINTER(C.c_void_p)), ("wdown_dev", C.POINTER(C.c_void_p)),
        ("g1_dev", C.POINTER(C.c_void_p)), ("g2_dev", C.POINTER(C.c_void_p)),
    ]


class KgDraftOut(C.Structure):
    _fields_ = [("n_drafted", C.c_int32), ("n_steps", C.c_int32),
                ("tokens", C.c_int32 * KG_GAMMA_MAX), ("conf", C.c_float * KG_GAMMA_MAX)]


class KgVerifyOut(C.Structure):
    _fields_ = [("n_rows", C.c_int32), ("n_accept", C.c_int32), ("n_emitted", C.c_int32),
                ("emitted", C.c_int32 * KG_M_MAX), ("target", C.c_int32 * KG_M_MAX)]


class KgStats(C.Structure):
    _fields_ = [("rounds", C.c_int32), ("tokens", C.c_int32), ("draft_steps", C.c_int32),
                ("drafted", C.c_int32), ("accepted", C.c_int32),
                ("cr", C.c_double), ("ctar", C.c_double * (KG_M_MAX + 1)), ("ms_decode", C.c_float)]


class KgError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        detail = ""
        if status in (KG_E_CUDA, KG_E_INTERNAL):
            detail = " [" + load().kg_last_cuda_error().decode() + "]"
        super().__init__(f"{what}: {status} ({strerror(status)}){detail}")


_lib = None


def load():
    """Loads libkangaroo.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: run `python -c 'import __graft_entry__ as g; g.build()'` first")
    lib = C.CDLL(path)
    vp, i32, u64, f32 = C.c_void_p, C.c_int32, C.c_uint64, C.c_float
    lib.kg_workspace_bytes.restype = C.c_size_t
    lib.kg_workspace_bytes.argtypes = [C.POINTER(KgConfig), C.c_int]
    lib.kg_init_model.argtypes = [C.POINTER(KgConfig), C.POINTER(KgWeights), vp, C.c_size_t, vp, C.POINTER(vp)]
    lib.kg_free_model.argtypes = [vp]
    lib.kg_reset.argtypes = [vp]
    lib.kg_prefill.argtypes = [vp, vp, i32, C.POINTER(i32)]
    lib.kg_prefill_device.argtypes = [vp, vp, i32]
    lib.kg_draft.argtypes = [vp, f32, i32, i32, C.POINTER(KgDraftOut)]
    lib.kg_verify.argtypes = [vp, C.POINTER(KgVerifyOut)]
    lib.kg_decode.argtypes = [vp, i32, f32, i32, i32, C.POINTER(KgStats)]
    lib.kg_decode_ar.argtypes = [vp, i32, vp]
    lib.kg_generate.argtypes = [vp, vp, i32, i32, f32, i32, i32, vp, C.POINTER(i32), C.POINTER(KgStats)]
    lib.kg_read_tokens.argtypes = [vp, vp, i32, C.POINTER(i32)]
    lib.kg_read_S.argtypes = [vp, vp, i32, C.POINTER(i32)]
    lib.kg_read_round_log.argtypes = [vp, vp, i32, C.POINTER(i32)]
    lib.kg_debug_logits.argtypes = [vp, i32, i32, vp]
    lib.kg_read_weight.argtypes = [vp, C.c_char_p, i32, u64, u64, vp]
    lib.kg_debug_fill_state.argtypes = [vp, i32, i32, u64]
    lib.kg_op_scratch_bytes.restype = C.c_size_t
    lib.kg_op_scratch_bytes.argtypes = []
    lib.kg_op_linear.argtypes = [i32, vp, vp, i32, i32, vp, i32, vp, f32, vp, i32, vp, vp, vp]
    lib.kg_op_lm_head.argtypes = [i32, vp, i32, i32, vp, i32, vp, f32, f32, vp, vp, vp, vp, vp]
    lib.kg_op_lm_head_noalloc.argtypes = [i32, vp, i32, i32, vp, i32, vp, f32, f32, vp, vp, vp, vp]
    lib.kg_op_attention.argtypes = [i32, vp, i32, i32, i32, i32, f32, vp, vp, vp, i32, vp, vp, vp]
    lib.kg_op_gemm.argtypes = [vp, i32, i32, vp, i32, vp, vp, vp, vp]
    lib.kg_strerror.restype = C.c_char_p
    lib.kg_strerror.argtypes = [C.c_int]
    lib.kg_last_cuda_error.restype = C.c_char_p
    lib.kg_last_cuda_error.argtypes = []
    lib.kg_debug_force_simple.argtypes = [vp, C.c_int]
    lib.kg_debug_force_simple_ops.argtypes = [C.c_int]
    lib.kg_debug_set_wait_budget.argtypes = [vp, C.c_double]
    lib.kg_debug_skip_barrier_arrival.argtypes = [vp, C.c_int]
    lib.kg_debug_set_prefill_mode.argtypes = [vp, C.c_int]
    _lib = lib
    return lib


def strerror(status: int) -> str:
    return load().kg_strerror(int(status)).decode()


def _check(status, what):
    if status != KG_OK:
        raise KgError(status, what)


def config_from_shape(shape, debug_logits=False, page_shuffle=False) -> KgConfig:
    """KgConfig from a shape object with the attribute names used by the input generator."""
    c = KgConfig()
    c.struct_size = C.sizeof(KgConfig)
    c.n_layers, c.d_model, c.n_heads, c.head_dim = shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim
    c.d_ffn, c.vocab, c.exit_layer = shape.d_ffn, shape.vocab, shape.exit_layer
    c.dtype = KG_BF16 if shape.dtype == "bf16" else KG_F32
    c.rms_eps, c.rope_theta, c.logit_scale = shape.rms_eps, shape.rope_theta, shape.logit_scale
    c.max_seq, c.page_size, c.gamma_max = shape.max_seq, shape.page_size, shape.gamma_max
    c.debug_logits, c.page_shuffle = int(debug_logits), int(page_shuffle)
    c.seed = shape.seed
    c.init_std, c.embed_std = shape.init_std, shape.embed_std
    c.deep_resid_scale, c.adapter_resid_scale, c.gain_std = shape.deep_resid_scale, shape.adapter_resid_scale, shape.gain_std
    return c


class KangarooModel:
    """A model living in a torch-owned device arena, driven through the C ABI."""

    def __init__(self, shape, debug_logits=False, page_shuffle=False, device="cuda:0", stream=None, weights=None,
                 arena=None):
        """weights: None (the library fills seeded synthetic weights into the arena) or the nested dict of host
        arrays the input generator makes; those are uploaded as torch tensors and handed over as borrowed
        pointers (kg_weights).  arena: an existing uint8 device tensor to build the model in."""
        import torch
        self.torch = torch
        self.lib = load()
        self.shape = shape
        self.cfg = config_from_shape(shape, debug_logits, page_shuffle)
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        nbytes = self.lib.kg_workspace_bytes(C.byref(self.cfg), 0 if weights is not None else 1)
        if nbytes == 0:
            raise KgError(KG_E_ARG, "kg_workspace_bytes")
        if arena is not None and arena.numel() < nbytes:
            raise KgError(KG_E_NOMEM, "arena")
        self.arena = arena if arena is not None else torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        kw = self._borrowed(weights) if weights is not None else None
        h = C.c_void_p()
        _check(self.lib.kg_init_model(C.byref(self.cfg), C.byref(kw) if kw is not None else None, self.arena.data_ptr(),
                                      self.arena.numel(), self.stream.cuda_stream, C.byref(h)), "kg_init_model")
        self.h = h
        self.arena_bytes = nbytes

    def _borrowed(self, w):
        """Uploads the host weights and returns the kg_weights table of device pointers (tensors kept alive here)."""
        torch = self.torch
        mdt = torch.bfloat16 if self.shape.dtype == "bf16" else torch.float32
        self._wt = []

        def up(a, dt):
            t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(self.device).to(dt).contiguous()
            self._wt.append(t)
            return t.data_ptr()

        L = self.shape.n_layers
        blocks = list(w["layers"]) + [w["adapter"]]
        kw = KgWeights()
        kw.embed_dev, kw.head_dev = up(w["embed"], mdt), up(w["head"], mdt)
        kw.g_final_dev = up(w["g_final"], torch.float32)

        def table(name, dt, adapter_name=None, with_adapter=True):
            arr = (C.c_void_p * (L + 1))()
            for i, blk in enumerate(blocks):
                if i == L and not with_adapter:
                    arr[i] = None
                else:
                    arr[i] = up(blk[adapter_name if (i == L and adapter_name) else name], dt)
            self._wt.append(arr)
            return arr

        kw.wqkv_dev, kw.wo_dev = table("wqkv", mdt), table("wo", mdt)
        kw.wgate_dev = table("wgate", mdt, with_adapter=False)
        kw.wup_dev = table("wup", mdt, with_adapter=False)
        kw.wdown_dev = table("wdown", mdt, with_adapter=False)
        kw.g1_dev = table("g1", torch.float32, adapter_name="g_in")
        kw.g2_dev = table("g2", torch.float32, adapter_name="g_last")
        return kw

    def close(self):
        if self.h:
            self.lib.kg_free_model(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        _check(self.lib.kg_reset(self.h), "kg_reset")

    def prefill(self, prompt) -> int:
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        x0 = C.c_int32()
        _check(self.lib.kg_prefill(self.h, p.ctypes.data, len(p), C.byref(x0)), "kg_prefill")
        return x0.value

    def prefill_device(self, prompt_dev):
        _check(self.lib.kg_prefill_device(self.h, prompt_dev.data_ptr(), prompt_dev.numel()), "kg_prefill_device")

    def draft(self, eta, gamma, stop_mode=STOP_KEEP, sync=True):
        out = KgDraftOut()
        _check(self.lib.kg_draft(self.h, eta, gamma, stop_mode, C.byref(out) if sync else None), "kg_draft")
        if not sync:
            return None
        return dict(n_drafted=out.n_drafted, n_steps=out.n_steps,
                    tokens=list(out.tokens[:out.n_drafted]), conf=list(out.conf[:out.n_steps]))

    def verify(self, sync=True):
        out = KgVerifyOut()
        _check(self.lib.kg_verify(self.h, C.byref(out) if sync else None), "kg_verify")
        if not sync:
            return None
        return dict(n_rows=out.n_rows, k=out.n_accept, emitted=list(out.emitted[:out.n_emitted]),
                    target=list(out.target[:out.n_rows]))

    @staticmethod
    def _stats(st: KgStats):
        return dict(rounds=st.rounds, tokens=st.tokens, draft_steps=st.draft_steps, drafted=st.drafted,
                    accepted=st.accepted, cr=st.cr, ctar=list(st.ctar), ms_decode=st.ms_decode)

    def decode(self, max_new, eta, gamma, stop_mode=STOP_KEEP, sync=True):
        st = KgStats()
        _check(self.lib.kg_decode(self.h, max_new, eta, gamma, stop_mode, C.byref(st) if sync else None), "kg_decode")
        return self._stats(st) if sync else None

    def decode_ar(self, n_tokens, sync=True):
        out = np.empty(n_tokens, dtype=np.int32)
        _check(self.lib.kg_decode_ar(self.h, n_tokens, out.ctypes.data if sync else None), "kg_decode_ar")
        return out.tolist() if sync else None

    def generate(self, prompt, max_new, eta, gamma, stop_mode=STOP_KEEP):
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        out = np.empty(max_new, dtype=np.int32)
        n = C.c_int32()
        st = KgStats()
        _check(self.lib.kg_generate(self.h, p.ctypes.data, len(p), max_new, eta, gamma, stop_mode,
                                    out.ctypes.data, C.byref(n), C.byref(st)), "kg_generate")
        return out[:n.value].tolist(), self._stats(st)

    def generate_into(self, prompt_host, out_host, max_new, eta, gamma, stop_mode=STOP_KEEP):
        """kg_generate on caller-owned host tensors (e.g. pinned torch int32 tensors): the prompt is read
        from prompt_host, the tokens are written to out_host.  Returns (n_out, stats)."""
        n = C.c_int32()
        st = KgStats()
        _check(self.lib.kg_generate(self.h, prompt_host.data_ptr(), prompt_host.numel(), max_new, eta, gamma, stop_mode,
                                    out_host.data_ptr(), C.byref(n), C.byref(st)), "kg_generate")
        return n.value, self._stats(st)

    def read_tokens(self, max_n=None):
        max_n = self.shape.max_seq + KG_M_MAX if max_n is None else max_n
        out = np.empty(max_n, dtype=np.int32)
        n = C.c_int32()
        _check(self.lib.kg_read_tokens(self.h, out.ctypes.data, max_n, C.byref(n)), "kg_read_tokens")
        return out[:n.value].tolist()

    def read_S(self, max_n=None):
        max_n = self.shape.max_seq + KG_M_MAX if max_n is None else max_n
        out = np.empty(max_n, dtype=np.int32)
        n = C.c_int32()
        _check(self.lib.kg_read_S(self.h, out.ctypes.data, max_n, C.byref(n)), "kg_read_S")
        return out[:n.value].tolist()

    def read_round_log(self, max_rounds=None):
        """One (n_d, n_steps, k, P) tuple per round run so far."""
        max_rounds = self.shape.max_seq + KG_M_MAX if max_rounds is None else max_rounds
        out = np.empty((max_rounds, 4), dtype=np.int32)
        n = C.c_int32()
        _check(self.lib.kg_read_round_log(self.h, out.ctypes.data, max_rounds, C.byref(n)), "kg_read_round_log")
        return [tuple(int(v) for v in row) for row in out[:n.value]]

    def debug_logits(self, which, row):
        out = np.empty(self.shape.vocab, dtype=np.float32)
        _check(self.lib.kg_debug_logits(self.h, which, row, out.ctypes.data), "kg_debug_logits")
        return out

    def read_weight(self, name, layer=0, offset=0, count=None):
        out = np.empty(count, dtype=np.float32)
        _check(self.lib.kg_read_weight(self.h, name.encode(), layer, offset, count, out.ctypes.data), "kg_read_weight")
        return out

    def fill_state(self, T, n_d, seed):
        _check(self.lib.kg_debug_fill_state(self.h, T, n_d, seed), "kg_debug_fill_state")

    def force_simple(self, on):
        _check(self.lib.kg_debug_force_simple(self.h, int(on)), "kg_debug_force_simple")

    def set_wait_budget(self, milliseconds):
        _check(self.lib.kg_debug_set_wait_budget(self.h, float(milliseconds)), "kg_debug_set_wait_budget")

    def set_prefill_mode(self, mode):
        _check(self.lib.kg_debug_set_prefill_mode(self.h, int(mode)), "kg_debug_set_prefill_mode")

    def skip_barrier_arrival(self, cta):
        _check(self.lib.kg_debug_skip_barrier_arrival(self.h, int(cta)), "kg_debug_skip_barrier_arrival")


# ---- single operators ---------------------------------------------------------------------------

def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream(torch):
    return torch.cuda.current_stream().cuda_stream


def op_scratch(torch, device="cuda:0"):
    return torch.empty(load().kg_op_scratch_bytes(), dtype=torch.uint8, device=device)


def op_linear(W, x, gain=None, eps=1e-6, resid=None, W2=None, scratch=None):
    import torch
    lib = load()
    N, K = W.shape
    M = x.shape[0]
    out = torch.empty(M, N, dtype=torch.float32, device=x.device)
    dt = KG_BF16 if W.dtype == torch.bfloat16 else KG_F32
    scratch = op_scratch(torch, x.device) if scratch is None else scratch
    _check(lib.kg_op_linear(dt, W.data_ptr(), _ptr(W2), N, K, x.data_ptr(), M, _ptr(gain), eps, _ptr(resid),
                            int(W2 is not None), out.data_ptr(), scratch.data_ptr(), _stream(torch)), "kg_op_linear")
    return out


def op_gemm(W, x, resid=None, scratch=None):
    import torch
    lib = load()
    N, K = W.shape
    M = x.shape[0]
    out = torch.empty(M, N, dtype=torch.float32, device=x.device)
    scratch = op_scratch(torch, x.device) if scratch is None else scratch
    _check(lib.kg_op_gemm(W.data_ptr(), N, K, x.data_ptr(), M, _ptr(resid), out.data_ptr(), scratch.data_ptr(), _stream(torch)), "kg_op_gemm")
    return out


def op_lm_head(W, x, gain, eps, logit_scale, want_logits=True, scratch=None):
    import torch
    lib = load()
    V, K = W.shape
    M = x.shape[0]
    tok = torch.empty(M, dtype=torch.int32, device=x.device)
    p = torch.empty(M, dtype=torch.float32, device=x.device)
    logits = torch.empty(M, V, dtype=torch.float32, device=x.device) if want_logits else None
    dt = KG_BF16 if W.dtype == torch.bfloat16 else KG_F32
    scratch = op_scratch(torch, x.device) if scratch is None else scratch
    _check(lib.kg_op_lm_head(dt, W.data_ptr(), V, K, x.data_ptr(), M, _ptr(gain), eps, logit_scale,
                             tok.data_ptr(), p.data_ptr(), _ptr(logits), scratch.data_ptr(), _stream(torch)), "kg_op_lm_head")
    return tok, p, logits


def op_lm_head_noalloc(W, x, gain, eps, logit_scale, tok, p, logits=None):
    """kg_op_lm_head_noalloc on caller-made tensors: tok (int32 [M]), p (float32 [M]) and optionally logits
    (float32 [M, V]) must exist already, so the call itself allocates nothing on the device."""
    import torch
    lib = load()
    V, K = W.shape
    M = x.shape[0]
    dt = KG_BF16 if W.dtype == torch.bfloat16 else KG_F32
    _check(lib.kg_op_lm_head_noalloc(dt, W.data_ptr(), V, K, x.data_ptr(), M, _ptr(gain), eps, logit_scale,
                                     tok.data_ptr(), p.data_ptr(), _ptr(logits), _stream(torch)), "kg_op_lm_head_noalloc")


def op_attention(qkv, pos0, n_heads, head_dim, rope_theta, kcache, vcache, page_table, page_size, scratch=None):
    import torch
    lib = load()
    M = qkv.shape[0]
    out = torch.empty(M, n_heads * head_dim, dtype=torch.float32, device=qkv.device)
    dt = KG_BF16 if kcache.dtype == torch.bfloat16 else KG_F32
    scratch = op_scratch(torch, qkv.device) if scratch is None else scratch
    _check(lib.kg_op_attention(dt, qkv.data_ptr(), M, pos0, n_heads, head_dim, rope_theta, kcache.data_ptr(),
                               vcache.data_ptr(), page_table.data_ptr(), page_size, out.data_ptr(),
                               scratch.data_ptr(), _stream(torch)), "kg_op_attention")
    return out
