"""Independent dense full-sequence forward in torch fp64, used ONLY to pin the oracle.

Written against torch's library routines (scaled_dot_product_attention, rms_norm,
silu, log_softmax, kl_div) and a complex-number form of the rotary embedding, so
that it shares neither code nor formulation with `oracle/surelock_oracle.py`
(numpy).  It knows nothing about locks, index lists or caches: it recomputes all
N rows ("the standard sampler recomputes every token each step", Sec. 2 of the
paper).  The one hook is `kv_override`, which replaces the K/V rows of chosen
positions before attention: the textbook statement of "locked positions are
attended through their cached K/V" (Sec. 2.1).
"""
import torch
import torch.nn.functional as F

D = torch.float64


def _rope_complex(x, theta):
    # x [N][H][dh]; pair (j, j+dh/2) seen as the complex number x_j + i x_{j+dh/2}, multiplied by e^{i pos theta_j}
    N, H, dh = x.shape
    half = dh // 2
    freqs = 1.0 / (theta ** (torch.arange(0, half, dtype=D) * 2.0 / dh))
    ang = torch.outer(torch.arange(N, dtype=D), freqs)
    rot = torch.polar(torch.ones_like(ang), ang)[:, None, :]
    z = torch.complex(x[..., :half], x[..., half:]) * rot
    return torch.cat([z.real, z.imag], dim=-1)


def dense_forward(cfg, w, tokens_1d, kv_override=None, return_kv=False):
    """Full forward of ONE sequence.  w: dict of torch fp64 tensors (same keys as the generators).

    kv_override: optional {layer: (positions LongTensor, K_rows [n][H][dh], V_rows)}.
    Returns logits [N][V] (and per-layer (K, V) [N][H][dh] when return_kv).
    """
    H, dh, d = cfg["n_heads"], cfg["head_dim"], cfg["d_model"]
    N = tokens_1d.shape[0]
    x = w["tok_emb"][tokens_1d.long()].to(D)
    kvs = []
    for l, lw in enumerate(w["layers"]):
        h = F.rms_norm(x, (d,), lw["attn_norm_g"].to(D), cfg["rms_eps"])
        q = _rope_complex(F.linear(h, lw["wq"].to(D)).view(N, H, dh), cfg["rope_theta"])
        k = _rope_complex(F.linear(h, lw["wk"].to(D)).view(N, H, dh), cfg["rope_theta"])
        v = F.linear(h, lw["wv"].to(D)).view(N, H, dh)
        if kv_override is not None and l in kv_override:
            p, ko, vo = kv_override[l]
            k = k.clone(); v = v.clone()
            k[p] = ko.to(D); v[p] = vo.to(D)
        kvs.append((k, v))
        o = F.scaled_dot_product_attention(q.transpose(0, 1), k.transpose(0, 1), v.transpose(0, 1))
        x = x + F.linear(o.transpose(0, 1).reshape(N, H * dh), lw["wo"].to(D))
        h2 = F.rms_norm(x, (d,), lw["ffn_norm_g"].to(D), cfg["rms_eps"])
        x = x + F.linear(F.silu(F.linear(h2, lw["w_gate"].to(D))) * F.linear(h2, lw["w_up"].to(D)),
                         lw["w_down"].to(D))
    logits = F.linear(F.rms_norm(x, (d,), w["final_norm_g"].to(D), cfg["rms_eps"]), w["lm_head"].to(D))
    if return_kv:
        return logits, kvs, x
    return logits


def kl_torch(logits_cur, logits_prev):
    """KL(p_cur || p_prev) per row via torch's kl_div (library routine)."""
    lp_cur = F.log_softmax(logits_cur.to(D), dim=-1)
    lp_prev = F.log_softmax(logits_prev.to(D), dim=-1)
    return F.kl_div(lp_prev, lp_cur, reduction="none", log_target=True).sum(-1)
