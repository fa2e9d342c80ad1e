"""A textbook causal transformer decoder, written separately from the oracle with torch
library routines (scaled_dot_product_attention, rms_norm, linear, embedding) in float64.

It knows nothing about subsequences, delay times or visibility rules: one token stream, a
lower-triangular mask, one position id per token.  The tests use it to pin the oracle in the
two cases where the pipelined decoder must reduce to ordinary causal decoding."""
import math

import torch
import torch.nn.functional as F


def t5_causal_buckets(dist: torch.Tensor, num_buckets: int, max_dist: int) -> torch.Tensor:
    """Bucket of a non-negative distance, vectorised the way the published T5 code does it."""
    exact = num_buckets // 2
    large = exact + (torch.log(dist.clamp(min=1).double() / exact) / math.log(max_dist / exact)
                     * (num_buckets - exact)).long()
    large = torch.minimum(large, torch.full_like(large, num_buckets - 1))
    return torch.where(dist < exact, dist, large)


def rope_complex(x: torch.Tensor, pos: torch.Tensor, theta: float) -> torch.Tensor:
    """Rotary embedding as a complex multiplication.  x [H, N, dh], pos [N]."""
    dh = x.shape[-1]
    freqs = theta ** (-torch.arange(0, dh, 2, dtype=torch.float64) / dh)
    rot = torch.polar(torch.ones(pos.shape[0], dh // 2, dtype=torch.float64), pos.double()[:, None] * freqs[None, :])
    xc = torch.view_as_complex(x.reshape(*x.shape[:-1], dh // 2, 2).contiguous())
    return torch.view_as_real(xc * rot[None]).reshape(x.shape)


def causal_decoder_logits(weights, hp, tokens, positions, enc_mem):
    """Logits [N, vocab] of a plain causal decoder over `tokens` with position ids `positions`."""
    W = {k: torch.as_tensor(v, dtype=torch.float64) for k, v in weights.items()}
    H, dh, L = hp["n_heads"], hp["d_head"], hp["n_layers"]
    hd = H * dh
    N = len(tokens)
    pos = torch.as_tensor(positions, dtype=torch.long)
    mem = torch.as_tensor(enc_mem, dtype=torch.float64)
    x = F.embedding(torch.as_tensor(tokens, dtype=torch.long), W["embed"])
    causal = torch.ones(N, N, dtype=torch.bool).tril()
    if hp["pos_mode"] == 0:
        dist = (pos[:, None] - pos[None, :]).clamp(min=0)
        bias = W["rel_bias"][:, t5_causal_buckets(dist, hp["rel_buckets"], hp["rel_max_dist"])]   # [H,N,N]
        attn_mask = bias.masked_fill(~causal[None], float("-inf"))
    else:
        attn_mask = torch.zeros(N, N, dtype=torch.float64).masked_fill(~causal, float("-inf"))[None]

    def heads(a):
        return a.reshape(a.shape[0], H, dh).transpose(0, 1)

    for l in range(L):
        h = F.rms_norm(x, (x.shape[-1],), W[f"l{l}.norm1"], hp["norm_eps"])
        q, k, v = F.linear(h, W[f"l{l}.wqkv"].T).split(hd, dim=-1)
        q, k, v = heads(q), heads(k), heads(v)
        if hp["pos_mode"] == 1:
            q, k = rope_complex(q, pos, hp["rope_theta"]), rope_complex(k, pos, hp["rope_theta"])
        a = F.scaled_dot_product_attention(q, k, v, attn_mask=attn_mask, scale=hp["attn_scale"])
        x = x + F.linear(a.transpose(0, 1).reshape(N, hd), W[f"l{l}.wo"].T)
        h = F.rms_norm(x, (x.shape[-1],), W[f"l{l}.norm2"], hp["norm_eps"])
        qc = heads(F.linear(h, W[f"l{l}.wq_c"].T))
        kc, vc = F.linear(mem, W[f"l{l}.wkv_c"].T).split(hd, dim=-1)
        c = F.scaled_dot_product_attention(qc, heads(kc), heads(vc), scale=hp["attn_scale"])
        x = x + F.linear(c.transpose(0, 1).reshape(N, hd), W[f"l{l}.wo_c"].T)
        h = F.rms_norm(x, (x.shape[-1],), W[f"l{l}.norm3"], hp["norm_eps"])
        x = x + F.linear(F.relu(F.linear(h, W[f"l{l}.w1"].T)), W[f"l{l}.w2"].T)
    return F.linear(F.rms_norm(x, (x.shape[-1],), W["final_norm"], hp["norm_eps"]), W["lm_head"]).numpy()
