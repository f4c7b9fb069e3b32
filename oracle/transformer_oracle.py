"""Slow, plain CPU oracle for the miss-path transformer layer and for the layer-wise caching loop.

TEST INFRASTRUCTURE ONLY: imported by the tests and by the benchmark's CPU legs; shares no code with the
CUDA path and never imports it.

What it computes:

* `layer_forward`: one transformer layer h_l = f_l(h_{l-1}) (Sec. IV-A of the paper calls it f_l and does
  not spell it out; it evaluates on BERT-base, DistilBERT and GPT-2 small, Sec. V-A).  This is the textbook
  layer: multi-head scaled dot-product self-attention, output projection, residual, layer normalisation,
  two-layer feed-forward network with GELU, residual, layer normalisation.  Two arrangements:
    post-norm, bidirectional, GELU with erf          (BERT-style encoder layer)
    pre-norm,  causal mask,  GELU with tanh formula  (GPT-2-style decoder layer)
* `embed`: h_0 = E(X), the hidden states that enter layer 1 in Algorithm 1: token embedding plus position
  embedding, followed (BERT-style embeddings) by a layer normalisation; the paper does not spell E out either.
* `infer`: Algorithm 1 (LLMCache-Infer) for a batch: for l = 1..L, probe bank l with the layer's input; hits
  take the stored output, misses run the layer and are inserted.

float64 arithmetic over the exact input values (weights and inputs are bf16 / f32 bit patterns).  With
`round_bf16=True` the intermediate tensors that the layer keeps in bf16 storage (q/k/v, attention output,
residual sums, normalised activations, FFN hidden) are rounded to bf16 at those points -- a storage-format
decision, like the bf16 bank -- so that the comparison with an implementation that stores them in bf16 is
tight; with False nothing is rounded.

Pins (tests/test_oracle_transformer.py): torch.nn.TransformerEncoderLayer in float64 (both arrangements),
torch.nn.functional.layer_norm / gelu, hand-worked softmax rows, the causal mask (a future token cannot
change an earlier output), permutation equivariance of the bidirectional layer, for `embed` a hand-worked row,
torch.nn.functional.embedding + layer_norm in float64, a table of zeros that leaves the position rows, and
an id outside the table; and for `infer` the chain
property of Algorithm 1 (a repeated input is served from the banks at every layer and returns the same bits).
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Optional

import numpy as np

from . import llmcache_oracle as O


@dataclass
class LayerWeights:
    """All matrices in [out_features, in_features] layout; bf16 bit patterns (uint16); vectors float32."""
    w_qkv: np.ndarray   # [3d, d]
    b_qkv: np.ndarray   # [3d]
    w_o: np.ndarray     # [d, d]
    b_o: np.ndarray     # [d]
    ln1_g: np.ndarray   # [d]
    ln1_b: np.ndarray
    w_1: np.ndarray     # [ffn, d]
    b_1: np.ndarray     # [ffn]
    w_2: np.ndarray     # [d, ffn]
    b_2: np.ndarray     # [d]
    ln2_g: np.ndarray
    ln2_b: np.ndarray


def _w(bits) -> np.ndarray:
    return O.bf16_to_f32(bits).astype(np.float64)


def _v(x) -> np.ndarray:
    return np.asarray(x, dtype=np.float32).astype(np.float64)


def _store(x: np.ndarray, round_bf16: bool) -> np.ndarray:
    if not round_bf16:
        return x
    return O.bf16_to_f32(O.bf16_round(x.astype(np.float32))).astype(np.float64)


def layer_norm(x: np.ndarray, g: np.ndarray, b: np.ndarray, eps: float = 1e-5) -> np.ndarray:
    """y = (x - mean) / sqrt(var + eps) * g + b over the last axis (biased variance)."""
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * g + b


def embed_f64(tokens: np.ndarray, tok_emb_bits: np.ndarray, pos_emb_bits: Optional[np.ndarray],
              layer_normed: bool = True, gain=None, bias=None, eps: float = 1e-5) -> np.ndarray:
    """h_0 = E(X) (Algorithm 1, the assignment before the loop) in float64, not rounded.

    tokens: int [S, n]; tok_emb_bits: bf16 bits [vocab, d]; pos_emb_bits: bf16 bits [n, d] or None.
    h_0[s, i] = E_tok[tokens[s, i]] + E_pos[i], then layer_norm over d if layer_normed (gain, bias: float32 [d],
    None = 1 and 0).  A token id outside the table gives a row of zeros.
    """
    tokens = np.asarray(tokens)
    S, n = tokens.shape
    E = _w(tok_emb_bits)
    vocab, d = E.shape
    out = np.zeros((S, n, d), dtype=np.float64)
    for s in range(S):
        for i in range(n):
            t = int(tokens[s, i])
            if t < 0 or t >= vocab:
                continue
            x = E[t].copy()
            if pos_emb_bits is not None:
                x = x + _w(pos_emb_bits[i])
            if layer_normed:
                g = np.ones(d) if gain is None else _v(gain)
                b = np.zeros(d) if bias is None else _v(bias)
                x = layer_norm(x, g, b, eps)
            out[s, i] = x
    return out


def embed(tokens, tok_emb_bits, pos_emb_bits, layer_normed=True, gain=None, bias=None, eps=1e-5) -> np.ndarray:
    """`embed_f64` stored as bf16 (round to nearest even): bit patterns [S, n, d]."""
    return O.bf16_round(embed_f64(tokens, tok_emb_bits, pos_emb_bits, layer_normed, gain, bias, eps).astype(np.float32))


_erf = np.vectorize(math.erf, otypes=[np.float64])


def gelu_erf(x: np.ndarray) -> np.ndarray:
    return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)))


def gelu_tanh(x: np.ndarray) -> np.ndarray:
    return 0.5 * x * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (x + 0.044715 * x ** 3)))


def attention(qkv: np.ndarray, heads: int, causal: bool) -> np.ndarray:
    """qkv [n, 3d] -> [n, d]: per head softmax(q k^T / sqrt(dh)) v; causal: position i sees j <= i."""
    n, d3 = qkv.shape
    d = d3 // 3
    dh = d // heads
    out = np.empty((n, d), dtype=np.float64)
    for h in range(heads):
        q = qkv[:, h * dh:(h + 1) * dh]
        k = qkv[:, d + h * dh:d + (h + 1) * dh]
        v = qkv[:, 2 * d + h * dh:2 * d + (h + 1) * dh]
        s = (q @ k.T) / math.sqrt(dh)
        if causal:
            s = np.where(np.tril(np.ones((n, n), dtype=bool)), s, -np.inf)
        s = s - s.max(axis=1, keepdims=True)
        p = np.exp(s)
        p = p / p.sum(axis=1, keepdims=True)
        out[:, h * dh:(h + 1) * dh] = p @ v
    return out


def layer_forward(x_bits: np.ndarray, w: LayerWeights, heads: int, pre_ln: bool = False, causal: bool = False,
                  tanh_gelu: bool = False, round_bf16: bool = False) -> np.ndarray:
    """One layer on one sequence.  x_bits: uint16 [n, d] (bf16).  Returns bf16 bit patterns [n, d]."""
    return O.bf16_round(layer_forward_f64(x_bits, w, heads, pre_ln, causal, tanh_gelu, round_bf16).astype(np.float32))


def layer_forward_f64(x_bits: np.ndarray, w: LayerWeights, heads: int, pre_ln: bool = False, causal: bool = False,
                      tanh_gelu: bool = False, round_bf16: bool = False) -> np.ndarray:
    """The layer's output before it is stored as bf16 (float64 [n, d])."""
    act = gelu_tanh if tanh_gelu else gelu_erf
    x = O.bf16_to_f32(x_bits).astype(np.float64)
    st = lambda t: _store(t, round_bf16)
    if not pre_ln:
        qkv = st(x @ _w(w.w_qkv).T + _v(w.b_qkv))
        a = st(attention(qkv, heads, causal))
        t = st(a @ _w(w.w_o).T + _v(w.b_o) + x)
        y = st(layer_norm(t, _v(w.ln1_g), _v(w.ln1_b)))
        f = st(act(y @ _w(w.w_1).T + _v(w.b_1)))
        t2 = st(f @ _w(w.w_2).T + _v(w.b_2) + y)
        out = layer_norm(t2, _v(w.ln2_g), _v(w.ln2_b))
    else:
        u = st(layer_norm(x, _v(w.ln1_g), _v(w.ln1_b)))
        qkv = st(u @ _w(w.w_qkv).T + _v(w.b_qkv))
        a = st(attention(qkv, heads, causal))
        x1 = st(a @ _w(w.w_o).T + _v(w.b_o) + x)
        v = st(layer_norm(x1, _v(w.ln2_g), _v(w.ln2_b)))
        f = st(act(v @ _w(w.w_1).T + _v(w.b_1)))
        out = f @ _w(w.w_2).T + _v(w.b_2) + x1
    return out


def infer(banks: List[O.Bank], layers: List[LayerWeights], h0_bits: np.ndarray, heads: int, pre_ln=False,
          causal=False, tanh_gelu=False, round_bf16=False, tau: Optional[float] = None):
    """Algorithm 1 for a batch.  h0_bits: uint16 [B, n, d].  Returns (h_L bits [B, n*d], hits per layer)."""
    B, n, d = h0_bits.shape
    h = h0_bits.reshape(B, n, d)
    hits = []
    for bank, w in zip(banks, layers):
        h_out = np.zeros((B, n * d), dtype=np.uint16)
        pr = O.probe(bank, h, "bf16", tau=tau, h_out=h_out)          # lookup; hits: h_l <- h'
        miss_out = np.zeros((len(pr.miss_idx), n * d), dtype=np.uint16)
        for m, b in enumerate(pr.miss_idx.tolist()):                 # misses: h_l <- f_l(h_{l-1})
            miss_out[m] = layer_forward(h[b], w, heads, pre_ln, causal, tanh_gelu, round_bf16).reshape(-1)
        O.commit(bank, pr, miss_out, h_out)                          # C_l[f_X] <- h_l
        hits.append(int(pr.hit.sum()))
        h = h_out.reshape(B, n, d)
    return h.reshape(B, n * d), hits


def divergence_check(bank: O.Bank, w: LayerWeights, h_bits: np.ndarray, pr: O.ProbeResult, heads: int,
                     stride: int, bound: float, pre_ln=False, causal=False, tanh_gelu=False, round_bf16=False):
    """Divergence monitor (Sec. III-E, divergence tracking of the outputs stored under a fingerprint;
    Sec. IV-D, the monitor that re-checks stored entries).  For every `stride`-th hit of the probe (in ascending batch
    order) the layer is recomputed on that sequence's input and compared with the stored output it was
    served: rel = ||f_l(h) - h'||_2 / ||f_l(h)||_2.  An entry whose rel exceeds `bound` is invalidated,
    unless it was (re)inserted during the current tick.  Returns (list of (b, slot, rel), number invalidated)."""
    checked, dropped = [], 0
    n, d = bank.seq_len, bank.d_model
    for i in range(0, len(pr.hit_idx), stride):
        b = int(pr.hit_idx[i])
        slot = int(pr.slot[b])
        fresh = O.bf16_to_f32(layer_forward(h_bits[b].reshape(n, d), w, heads, pre_ln, causal, tanh_gelu,
                                            round_bf16)).astype(np.float64).reshape(-1)
        stored = O.bf16_to_f32(bank.act[slot % bank.act_rows]).astype(np.float64)
        den = float(np.sqrt(np.sum(fresh * fresh)))
        rel = float(np.sqrt(np.sum((fresh - stored) ** 2))) / den if den > 0 else 0.0
        checked.append((b, slot, rel))
        if rel > bound and bank.valid[slot] and int(bank.insert_tick[slot]) != bank.tick:
            bank.valid[slot] = 0
            dropped += 1
    return checked, dropped
