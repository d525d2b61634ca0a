"""CPU oracle for the DART draft forward pass -- TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 statement of what Section 3.2 ("Diffusion-Inspired Drafting Phase")
defines: fused target features + shifted token embedding -> one decoder layer over the
prefix KV cache plus K query rows -> own LM head -> one logit row per future position,
followed by Algorithm 1 lines 6-8 (top-k candidates and s_logit = log(softmax + eps),
Appendix D).  Only tests, the smoke check and the benchmark's CPU-baseline leg may call
this; the CUDA library never does and shares no code with it.

Inputs are the bf16 bit patterns (numpy uint16) that the library receives, widened
exactly; every operation after that is fp64 with no intermediate rounding.  numpy's
matmul is used as a library primitive for the contractions; nothing is blocked, fused
or reordered beyond chunking a weight matrix by rows to bound memory.

Where the paper is silent (norm placement, RoPE variant, mask-row representation ...)
the readings listed in the repository's design notes are used; each is marked "reading".
"""
from __future__ import annotations

import math
from typing import Dict, Optional

import numpy as np

from . import philox as _philox


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp64."""
    b = np.ascontiguousarray(bits).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp64 -> fp32 -> bf16 (nearest-even); used only for the cache append side effect."""
    f = np.ascontiguousarray(x, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def rmsnorm(x: np.ndarray, gamma: np.ndarray, eps: float) -> np.ndarray:
    """RMSNorm over the last axis: x * gamma / sqrt(mean(x^2) + eps)  (reading: Qwen3-style)."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x * gamma / np.sqrt(ms + eps)


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding, rotate-half pairing (i, i + d_h/2), angle = pos * theta^(-2i/d_h).

    x: [..., rows, d_h]; pos: [rows] absolute positions  (Appendix B: Q,K rotated by position ids).
    """
    dh = x.shape[-1]
    half = dh // 2
    inv = theta ** (-(2.0 * np.arange(half, dtype=np.float64)) / dh)
    ang = pos.astype(np.float64)[:, None] * inv[None, :]
    c, s = np.cos(ang), np.sin(ang)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def linear(x: np.ndarray, w_bits: np.ndarray, row_chunk: int = 8192) -> np.ndarray:
    """y = x @ W^T with W given as bf16 bits [out, in]; widened chunk by chunk."""
    out_dim = w_bits.shape[0]
    y = np.empty(x.shape[:-1] + (out_dim,), dtype=np.float64)
    for s in range(0, out_dim, row_chunk):
        e = min(out_dim, s + row_chunk)
        y[..., s:e] = x @ bf16_to_f64(w_bits[s:e]).T
    return y


def visible(P: int, r: int, s: int) -> bool:
    """Causal rule of Section 3.1: query row r (absolute position P+r) sees key position s
    iff s <= P + r -- every cached prefix position and the new rows up to itself."""
    return s <= P + r


def attention_rows(q: np.ndarray, k_all: np.ndarray, v_all: np.ndarray, P: int) -> np.ndarray:
    """softmax(q k^T / sqrt(d_h)) v for one sequence with grouped-query heads.

    q: [K, H_q, d_h]; k_all, v_all: [H_kv, P + K, d_h] (cache rows 0..P-1 then the K new rows).
    Head j reads KV head j // (H_q / H_kv)  (Appendix B listing: grouped-query attention).
    """
    K, Hq, dh = q.shape
    Hkv = k_all.shape[0]
    G = Hq // Hkv
    out = np.zeros((K, Hq, dh), dtype=np.float64)
    scale = 1.0 / math.sqrt(dh)
    for j in range(Hq):
        kk, vv = k_all[j // G], v_all[j // G]
        for r in range(K):
            n_vis = P + r + 1                      # positions s with visible(P, r, s)
            sc = (kk[:n_vis] @ q[r, j]) * scale
            sc = sc - sc.max()
            p = np.exp(sc)
            p = p / p.sum()
            out[r, j] = p @ vv[:n_vis]
    return out


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def draft_forward(cfg: Dict, w: Dict[str, np.ndarray], inp: Dict[str, np.ndarray],
                  keep_intermediates: bool = False) -> Dict[str, np.ndarray]:
    """One drafting forward pass (Section 3.2) for a batch of independent sequences.

    cfg keys: hidden, n_q_heads, n_kv_heads, head_dim, K, rope_theta, rms_eps.
    w: bf16 bit arrays (uint16) -- w_fc [h,3h], embed [V,h], mask_vec [2h], norm_g, norm_e,
       w_q [Hq*dh,2h], w_k, w_v [Hkv*dh,2h], w_o [h,Hq*dh], norm_post, w_gate, w_up [I,h],
       w_down [h,I], norm_final, w_lm [V,h].
    inp: feats bits [B,F,3h], tokens [B,F], seq_lens [B], k_cache/v_cache bits [B,Hkv,Pcap,dh],
       n_fresh F.  n_fresh may also be a sequence of B per-sequence counts F_b (the steady-state call after a
       verification that accepted a different number of tokens per sequence, Section 3.2 / Figure 2); the
       fresh rows' features and tokens are then packed in sequence order: feats [sum F_b, 3h], tokens [sum F_b].
    Returns logits [B,K,V] (row r predicts the token after absolute position P_b + r: shifted
    logits, Section 3.2) and the new rows' post-RoPE k and v [B,K,Hkv,dh].
    """
    h, Hq, Hkv, dh, K = (cfg[n] for n in ("hidden", "n_q_heads", "n_kv_heads", "head_dim", "K"))
    theta, eps = float(cfg["rope_theta"]), float(cfg["rms_eps"])
    seq_lens = np.asarray(inp["seq_lens"]).astype(np.int64)
    B = seq_lens.shape[0]
    Fb = np.broadcast_to(np.asarray(inp["n_fresh"], dtype=np.int64), (B,))      # fresh rows of each sequence
    gam = {n: bf16_to_f64(w[n]) for n in ("norm_g", "norm_e", "norm_post", "norm_final")}
    m = bf16_to_f64(w["mask_vec"])

    # rows r < F carry fresh target features; the others are <mask> rows (reading: one learned
    # 2h-vector stands in for the pre-norm [g ; e] of every mask row)
    g = np.empty((B, K, h), dtype=np.float64)
    e = np.empty((B, K, h), dtype=np.float64)
    if Fb.sum() > 0:
        if w.get("w_fc") is None:                               # the caller fused the features itself: feats = g [.., h]
            gf = bf16_to_f64(inp["feats"]).reshape(-1, h)
        else:
            feats = bf16_to_f64(inp["feats"]).reshape(-1, 3 * h)    # fresh rows packed in sequence order
            gf = linear(feats, w["w_fc"])                           # fused features, no bias (reading)
        ef = bf16_to_f64(w["embed"][np.asarray(inp["tokens"]).astype(np.int64).reshape(-1)])  # shifted embedding
    off = 0
    for b in range(B):
        F = int(Fb[b])
        g[b, :F] = gf[off:off + F] if F else 0.0
        e[b, :F] = ef[off:off + F] if F else 0.0
        g[b, F:] = m[:h]
        e[b, F:] = m[h:]
        off += F
    z = np.concatenate([rmsnorm(g, gam["norm_g"], eps), rmsnorm(e, gam["norm_e"], eps)], axis=-1)
    res = g                                                     # residual = un-normed g (reading)

    q = linear(z, w["w_q"]).reshape(B, K, Hq, dh)
    kn = linear(z, w["w_k"]).reshape(B, K, Hkv, dh)
    vn = linear(z, w["w_v"]).reshape(B, K, Hkv, dh)
    attn = np.empty((B, K, Hq * dh), dtype=np.float64)
    for b in range(B):
        P = int(seq_lens[b])
        pos = P + np.arange(K)
        qb = rope(q[b].transpose(1, 0, 2), pos, theta).transpose(1, 0, 2)     # [K,Hq,dh]
        kb = rope(kn[b].transpose(1, 0, 2), pos, theta)                        # [Hkv,K,dh]
        kn[b] = kb.transpose(1, 0, 2)
        q[b] = qb
        k_all = np.concatenate([bf16_to_f64(inp["k_cache"][b, :, :P]), kb], axis=1)
        v_all = np.concatenate([bf16_to_f64(inp["v_cache"][b, :, :P]), vn[b].transpose(1, 0, 2)], axis=1)
        attn[b] = attention_rows(qb, k_all, v_all, P).reshape(K, Hq * dh)

    x1 = res + linear(attn, w["w_o"])
    n2 = rmsnorm(x1, gam["norm_post"], eps)
    u = silu(linear(n2, w["w_gate"])) * linear(n2, w["w_up"])
    x2 = x1 + linear(u, w["w_down"])
    n3 = rmsnorm(x2, gam["norm_final"], eps)
    logits = linear(n3, w["w_lm"], row_chunk=4096)
    out = {"logits": logits, "k_new": kn, "v_new": vn}
    if keep_intermediates:
        out.update(g=g, e=e, z=z, q=q, attn=attn, x1=x1, n2=n2, u=u, x2=x2, n3=n3)
    return out


def prefill_kv(cfg: Dict, w: Dict[str, np.ndarray], feats: np.ndarray, tokens: np.ndarray, positions: np.ndarray):
    """Keys and values of the draft layer for new prefix rows (Section 3.2: the layer attends over its own KV
    cache of the prefix).  A single layer's k and v depend on the layer's input alone, so no attention is needed:
    row i with target features feats[i] (bf16 bits [n, 3h]), next-token id tokens[i] and absolute position
    positions[i] gives z = [RMSNorm(W_fc f) ; RMSNorm(E[token])], k = RoPE(W_k z, position), v = W_v z.
    Returns k, v as fp64 [n, Hkv, dh]."""
    h, Hkv, dh = cfg["hidden"], cfg["n_kv_heads"], cfg["head_dim"]
    theta, eps = float(cfg["rope_theta"]), float(cfg["rms_eps"])
    g = linear(bf16_to_f64(feats).reshape(-1, 3 * h), w["w_fc"])
    e = bf16_to_f64(w["embed"][np.asarray(tokens).astype(np.int64).reshape(-1)])
    z = np.concatenate([rmsnorm(g, bf16_to_f64(w["norm_g"]), eps), rmsnorm(e, bf16_to_f64(w["norm_e"]), eps)], axis=-1)
    n = z.shape[0]
    k = linear(z, w["w_k"]).reshape(n, Hkv, dh)
    v = linear(z, w["w_v"]).reshape(n, Hkv, dh)
    pos = np.asarray(positions).astype(np.int64)
    k = rope(k.transpose(1, 0, 2), pos, theta).transpose(1, 0, 2)
    return k, v


def log_softmax(y: np.ndarray) -> np.ndarray:
    mx = y.max(axis=-1, keepdims=True)
    return y - (mx + np.log(np.sum(np.exp(y - mx), axis=-1, keepdims=True)))


def gumbel_noise(vocab: int, row: int, b: int, step: int, seed: int) -> np.ndarray:
    """Gumbel(0,1) noise for every vocab id of one logit row (reading of T > 0 drafting:
    Gumbel-top-k = k draws without replacement from the softmax).  The 32-bit integer for
    token v is word v & 3 of Philox4x32-10(counter=(v>>2, row, b, step), key=seed), mapped to
    u = ((x >> 8) + 0.5) * 2^-24 and G = -log(-log u)."""
    nblk = (vocab + 3) // 4
    ctr = np.zeros((nblk, 4), dtype=np.uint32)
    ctr[:, 0] = np.arange(nblk, dtype=np.uint32)
    ctr[:, 1] = np.uint32(row)
    ctr[:, 2] = np.uint32(b)
    ctr[:, 3] = np.uint32(step & 0xFFFFFFFF)
    key = (np.uint32(seed & 0xFFFFFFFF), np.uint32((seed >> 32) & 0xFFFFFFFF))
    x = _philox.philox4x32_10(ctr, key).reshape(-1)[:vocab]
    u = ((x >> np.uint32(8)).astype(np.float64) + 0.5) * (2.0 ** -24)
    return -np.log(-np.log(u))


def topk_candidates(logits_row: np.ndarray, k: int, eps_logit: float, temperature: float = 0.0,
                    noise: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Algorithm 1 lines 6-8 for one position: S_i = top-k tokens, s_logit = log(softmax + eps).

    Order: selection value descending, ties to the lower token id (reading).  With
    temperature > 0 the selection value is y + Gumbel noise while s_logit stays the
    un-perturbed log(softmax(y) + eps), y = logits / T.
    """
    y = logits_row / temperature if temperature > 0 else logits_row
    lp = log_softmax(y)
    sel = y + noise if (temperature > 0 and noise is not None) else y
    k = min(k, y.shape[-1])
    order = np.lexsort((np.arange(y.shape[-1]), -sel))[:k]
    return {"ids": order.astype(np.int32), "slogit": np.log(np.exp(lp[order]) + eps_logit),
            "lp": lp, "sel": sel}
