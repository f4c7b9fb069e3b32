"""Seeded synthetic inputs shaped like the paper's BERT / GPT-2 workloads.

The paper evaluates on WikiText-103, SQuAD v2 and OpenBookQA through
pretrained BERT-base, DistilBERT and GPT-2 small (Sec. V-A); neither the data
nor the weights are used here.  These generators produce inputs with the same
shapes (d_model 768 / 1024, sequence lengths 128 ... 1024, vocabulary sizes,
bank sizes) and with a controlled similarity structure (cluster centres, near
duplicates, token-level edits, shared prefixes).

Nothing in this module implements any step of the method: it only draws
random tensors.  Every function is a pure function of its seed and device;
the same tensor bytes are then handed to whichever implementation consumes
them.
"""
from __future__ import annotations

import torch

BASE_SEED = 20251216


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def randn(shape, seed, device="cpu", dtype=torch.float32, scale=1.0):
    x = torch.randn(shape, generator=_gen(seed, device), device=device, dtype=torch.float32)
    if scale != 1.0:
        x = x * scale
    return x.to(dtype)


def bf16_bits(t: torch.Tensor):
    """uint16 numpy view of a bf16 tensor's bit patterns (host copy)."""
    return t.detach().to("cpu").contiguous().view(torch.int16).numpy().view("uint16")


def from_bf16_bits(bits, device="cpu") -> torch.Tensor:
    import numpy as np
    return torch.from_numpy(np.ascontiguousarray(bits).view("int16").copy()).view(torch.bfloat16).to(device)


# ---------------------------------------------------------------------------
# Cluster workload (single-layer probe and the drifting-centre churn):
# hidden states = centre tensor + per-element Gaussian noise.
# ---------------------------------------------------------------------------
class ClusterWorkload:
    """`n_centres` centre tensors [n, d] ~ N(0,1); entries and queries are noisy copies."""

    def __init__(self, n_centres, seq_len, d_model, seed=BASE_SEED, device="cpu", dtype=torch.float32):
        self.n, self.d, self.device, self.dtype, self.seed = seq_len, d_model, device, dtype, seed
        self.centres = randn((n_centres, seq_len, d_model), seed, device)

    def entries(self, first, count, sigma=0.05):
        """Hidden states of bank entries first..first+count-1; entry i belongs to centre i mod n_centres."""
        idx = torch.arange(first, first + count, device=self.device) % self.centres.shape[0]
        noise = randn((count, self.n, self.d), self.seed + 7919 * (first + 1), self.device, scale=sigma)
        return (self.centres[idx] + noise).to(self.dtype)

    def queries(self, count, n_entries, seed, sigma=0.05, near_fraction=0.5, entry_sigma=0.05):
        """`near_fraction` of the queries = a seeded random bank entry + fresh noise (expected hits),
        the rest fresh N(0,1) (expected misses); shuffled.  Returns (h, source_entry) with -1 for fresh."""
        g = _gen(seed, self.device)
        n_near = int(round(count * near_fraction))
        src = torch.randint(0, n_entries, (n_near,), generator=g, device=self.device)
        h = torch.empty((count, self.n, self.d), dtype=torch.float32, device=self.device)
        for i in range(n_near):                      # regenerate the chosen entries one by one
            e = int(src[i])
            h[i] = self.entries(e, 1, entry_sigma)[0].float()
        h[:n_near] += torch.randn((n_near, self.n, self.d), generator=g, device=self.device) * sigma
        h[n_near:] = torch.randn((count - n_near, self.n, self.d), generator=g, device=self.device)
        source = torch.full((count,), -1, dtype=torch.int64, device=self.device)
        source[:n_near] = src
        perm = torch.randperm(count, generator=g, device=self.device)
        return h[perm].to(self.dtype).contiguous(), source[perm]


def activations(count, seq_len, d_model, seed, device="cpu"):
    """Stand-in layer outputs (content is irrelevant to the probe): bf16 [count, n*d]."""
    return randn((count, seq_len * d_model), seed, device, dtype=torch.bfloat16)


def projection(d_model, fp_dim, seed, device="cpu"):
    """Seeded Gaussian N(0, 1/k) matrix [d, k] in bf16: random hyperplanes standing in for PCA loadings."""
    return randn((d_model, fp_dim), seed, device, dtype=torch.bfloat16, scale=fp_dim ** -0.5)


# ---------------------------------------------------------------------------
# Token workloads (BERT-base- and GPT-2-small-shaped): embedding-level hidden
# states h0 = LayerNorm(E[token] + P[position]) with E, P ~ N(0, 0.02^2).
# ---------------------------------------------------------------------------
class TokenWorkload:
    def __init__(self, vocab, seq_len, d_model, seed=BASE_SEED, device="cpu"):
        self.vocab, self.n, self.d, self.device, self.seed = vocab, seq_len, d_model, device, seed
        self.E = randn((vocab, d_model), seed + 1, device, dtype=torch.bfloat16, scale=0.02)
        self.P = randn((seq_len, d_model), seed + 2, device, dtype=torch.bfloat16, scale=0.02)

    def tokens(self, count, seed):
        return torch.randint(0, self.vocab, (count, self.n), generator=_gen(seed, self.device), device=self.device)

    def edited(self, seeds_tok, count, frac, seed):
        """`count` copies of the seed sequences (round robin) with `frac` of positions resampled."""
        g = _gen(seed, self.device)
        S = seeds_tok.shape[0]
        src = torch.arange(count, device=self.device) % S
        tok = seeds_tok[src].clone()
        n_edit = int(round(self.n * frac))
        for i in range(count):
            pos = torch.randperm(self.n, generator=g, device=self.device)[:n_edit]
            tok[i, pos] = torch.randint(0, self.vocab, (n_edit,), generator=g, device=self.device)
        return tok, src

    def with_shared_prefix(self, seeds_tok, count, prefix_len, seed):
        """Sequence i = first prefix_len tokens of seed i mod S, then uniform random tokens."""
        g = _gen(seed, self.device)
        S = seeds_tok.shape[0]
        src = torch.arange(count, device=self.device) % S
        tok = torch.randint(0, self.vocab, (count, self.n), generator=g, device=self.device)
        tok[:, :prefix_len] = seeds_tok[src, :prefix_len]
        return tok, src

    def hidden(self, tok, chunk=32):
        """bf16 [B, n, d] embedding-level hidden states of token sequences."""
        out = torch.empty((tok.shape[0], self.n, self.d), dtype=torch.bfloat16, device=self.device)
        for i in range(0, tok.shape[0], chunk):
            x = self.E[tok[i:i + chunk]].float() + self.P[None].float()
            out[i:i + chunk] = torch.nn.functional.layer_norm(x, (self.d,)).to(torch.bfloat16)
        return out


def shuffled(count, seed, device="cpu"):
    return torch.randperm(count, generator=_gen(seed, device), device=device)


# ---------------------------------------------------------------------------
# Fingerprint-level workload (bank-scan stress): keys and queries are drawn
# directly in fingerprint space.
# ---------------------------------------------------------------------------
def scan_stress(n_bank, n_query, k, n_clusters=4096, spread=0.1, near_fraction=0.3, q_sigma=0.05,
                seed=BASE_SEED, device="cpu", chunk=65536):
    """Returns (bank bf16 [n_bank,k] unit rows, queries bf16 [n_query,k], source int64 [n_query] or -1).
    bank[i] = normalised(centre[i mod n_clusters] + spread*N(0,1)); near queries = a random bank row's
    unrounded vector + q_sigma*N(0,1); the rest fresh N(0,1)."""
    centres = randn((n_clusters, k), seed, device)
    bank = torch.empty((n_bank, k), dtype=torch.bfloat16, device=device)

    def rows(first, count):
        idx = torch.arange(first, first + count, device=device) % n_clusters
        return centres[idx] + randn((count, k), seed + 104729 * (first // chunk + 1), device, scale=spread)

    for f in range(0, n_bank, chunk):
        c = min(chunk, n_bank - f)
        r = rows(f, c)
        bank[f:f + c] = (r / r.norm(dim=1, keepdim=True)).to(torch.bfloat16)
    g = _gen(seed + 5, device)
    n_near = int(round(n_query * near_fraction))
    src = torch.randint(0, n_bank, (n_near,), generator=g, device=device)
    q = torch.randn((n_query, k), generator=g, device=device)
    # rebuild the unrounded source rows chunk by chunk
    for f in range(0, n_bank, chunk):
        c = min(chunk, n_bank - f)
        sel = ((src >= f) & (src < f + c)).nonzero().flatten()
        if sel.numel():
            r = rows(f, c)
            q[sel] = r[src[sel] - f] + q[sel] * q_sigma
    source = torch.full((n_query,), -1, dtype=torch.int64, device=device)
    source[:n_near] = src
    perm = torch.randperm(n_query, generator=g, device=device)
    return bank, q[perm].to(torch.bfloat16).contiguous(), source[perm]


def layer_weights(d_model, ffn, seed, device="cpu"):
    """Random-init transformer layer weights: bf16 matrices in [out, in] layout ~ N(0, 0.02^2) (the usual
    initialisation of BERT / GPT-2), f32 biases ~ N(0, 0.02^2), layer-norm gains 1 + N(0, 0.02^2)."""
    mat = lambda o, i, s: randn((o, i), seed + s, device, dtype=torch.bfloat16, scale=0.02)
    vec = lambda n, s, base=0.0: (randn((n,), seed + s, device, scale=0.02) + base).contiguous()
    return {"w_qkv": mat(3 * d_model, d_model, 1), "b_qkv": vec(3 * d_model, 2), "w_o": mat(d_model, d_model, 3),
            "b_o": vec(d_model, 4), "ln1_g": vec(d_model, 5, 1.0), "ln1_b": vec(d_model, 6),
            "w_1": mat(ffn, d_model, 7), "b_1": vec(ffn, 8), "w_2": mat(d_model, ffn, 9), "b_2": vec(d_model, 10),
            "ln2_g": vec(d_model, 11, 1.0), "ln2_b": vec(d_model, 12)}
