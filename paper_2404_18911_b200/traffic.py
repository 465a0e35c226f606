"""Algorithmic HBM bytes of the decode step's passes, from the model shape alone.

Host-side bookkeeping for roofline figures: every weight byte of the layers a pass touches is
counted once, plus the K/V entries the pass attends to and the K/V rows it writes.  Activations
(a few rows of d floats per operator) and norm gains are left out; they are below 0.1 % of any pass.
"""
from __future__ import annotations


def _es(shape) -> int:
    return 2 if shape.dtype == "bf16" else 4


def layer_weight_bytes(shape) -> int:
    d, F = shape.d_model, shape.d_ffn
    return (4 * d * d + 3 * d * F) * _es(shape)


def adapter_weight_bytes(shape) -> int:
    return 4 * shape.d_model * shape.d_model * _es(shape)


def head_weight_bytes(shape) -> int:
    return shape.vocab * shape.d_model * _es(shape)


def kv_bytes_per_token_layer(shape) -> int:
    return 2 * shape.d_model * _es(shape)


def _attn_kv_bytes(shape, n_layers: int, pos0: int, M: int) -> int:
    """K/V read (keys 0 .. pos0+M-1, once for all M rows) plus the M rows written, over n_layers."""
    return n_layers * (pos0 + M + M) * kv_bytes_per_token_layer(shape)


def shallow_pass_bytes(shape, pos: int) -> int:
    """Layers 1..l on one row at position pos (one early feature)."""
    l = shape.exit_layer
    return l * layer_weight_bytes(shape) + _attn_kv_bytes(shape, l, pos, 1) + shape.d_model * _es(shape)


def adapter_head_bytes(shape, pos0: int, M: int) -> int:
    """Adapter on M rows (1, or 2 when its cache lags) at pos0.. plus the shared LM head on the last row."""
    return adapter_weight_bytes(shape) + head_weight_bytes(shape) + _attn_kv_bytes(shape, 1, pos0, M)


def draft_step_bytes(shape, pos: int) -> int:
    """One full draft step: shallow pass + adapter + LM head, all on one row at position pos."""
    return shallow_pass_bytes(shape, pos) + adapter_head_bytes(shape, pos, 1)


def verify_bytes(shape, pos0: int, M: int) -> int:
    """Layers l+1..L on M rows at pos0.. plus the LM head."""
    n = shape.n_layers - shape.exit_layer
    return n * layer_weight_bytes(shape) + head_weight_bytes(shape) + _attn_kv_bytes(shape, n, pos0, M)


def ar_step_bytes(shape, pos: int) -> int:
    L = shape.n_layers
    return L * layer_weight_bytes(shape) + head_weight_bytes(shape) + _attn_kv_bytes(shape, L, pos, 1) + shape.d_model * _es(shape)


def round_bytes(shape, n_d: int, n_steps: int, P: int, len_A_lag: int = 0) -> int:
    """One Kangaroo round that kept n_d drafts after n_steps adapter+head passes, x_0 at position P:
    n_d+1 shallow passes, n_steps adapter+head passes, one verify pass on n_d+1 rows."""
    b = 0
    for j in range(n_d + 1):
        b += shallow_pass_bytes(shape, P + j)
    for j in range(n_steps):
        lag = len_A_lag if j == 0 else 0
        b += adapter_head_bytes(shape, P + j - lag, 1 + lag)
    b += verify_bytes(shape, P, n_d + 1)
    return b


def decode_bytes(shape, round_log) -> int:
    """Total over the rounds of a decode launch; round_log holds (n_d, n_steps, k, P) per round."""
    total = 0
    prev = None
    for (n_d, n_steps, k, P) in round_log:
        # the adapter cache lags by one position after a round whose drafts were all accepted
        # while the adapter had not seen the last early feature
        lag = 0
        if prev is not None:
            pn_d, pn_steps, pk, _ = prev
            lag = 1 if (pk == pn_d and pn_steps == pn_d) else 0
        total += round_bytes(shape, n_d, n_steps, P, lag)
        prev = (n_d, n_steps, k, P)
    return total


def prefill_bytes_chunked(shape, n: int, chunk: int) -> int:
    """Prefill as passes of `chunk` rows through every layer (weights re-read once per chunk)."""
    L = shape.n_layers
    total = 0
    for c0 in range(0, n, chunk):
        M = min(chunk, n - c0)
        total += L * layer_weight_bytes(shape) + adapter_weight_bytes(shape) * 3 // 4 + _attn_kv_bytes(shape, L + 1, c0, M)
    return total + head_weight_bytes(shape)
