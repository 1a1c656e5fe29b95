"""Pins for the oracle's cache-free model forward (oracle/model_oracle.py)."""
import numpy as np
import torch

from oracle import model_oracle as mo
from oracle import wedlm_oracle as orc
from workloads.model import TINY, make_model, make_prompts_and_targets


def _torch_reference_logits(w, m, tokens):
    """An independent float64 implementation from library pieces: torch SDPA with is_causal, F.silu,
    complex-number RoPE.  Plain causal decoder over `tokens` at positions 0..N-1."""
    t = {k: torch.tensor(orc.to_f64(v)) for k, v in w.items()}
    N = len(tokens)
    h = t["embed"][torch.tensor(tokens)]
    D = m.head_dim
    ang = torch.arange(N, dtype=torch.float64)[:, None] * (m.rope_theta ** (-2.0 * torch.arange(D // 2, dtype=torch.float64) / D))
    rot = torch.polar(torch.ones_like(ang), ang)                     # e^{i angle}

    def rope(x):                                                      # x [N, H, D], pairs (d, d + D/2)
        z = torch.complex(x[..., : D // 2], x[..., D // 2:]) * rot[:, None, :]
        return torch.cat([z.real, z.imag], dim=-1)

    def rms(x, g):
        return x * torch.rsqrt(x.pow(2).mean(-1, keepdim=True) + m.rms_eps) * g

    for l in range(m.n_layers):
        a = rms(h, t[f"l{l}.norm1"])
        q = rope((a @ t[f"l{l}.wq"]).view(N, m.n_q_heads, D))
        k = rope((a @ t[f"l{l}.wk"]).view(N, m.n_kv_heads, D))
        v = (a @ t[f"l{l}.wv"]).view(N, m.n_kv_heads, D)
        G = m.n_q_heads // m.n_kv_heads
        o = torch.nn.functional.scaled_dot_product_attention(
            q.permute(1, 0, 2)[None], k.repeat_interleave(G, dim=1).permute(1, 0, 2)[None],
            v.repeat_interleave(G, dim=1).permute(1, 0, 2)[None], is_causal=True)[0].permute(1, 0, 2)
        h = h + o.reshape(N, -1) @ t[f"l{l}.wo"]
        mm = rms(h, t[f"l{l}.norm2"])
        h = h + (torch.nn.functional.silu(mm @ t[f"l{l}.wg"]) * (mm @ t[f"l{l}.wu"])) @ t[f"l{l}.wd"]
    return (rms(h, t["norm_f"]) @ t["lm_head"]).numpy()


def test_filled_window_in_logical_order_is_a_plain_causal_decoder():
    w = make_model(TINY)
    toks = np.random.default_rng(0).integers(0, TINY.vocab - 1, size=15).tolist()
    ref = _torch_reference_logits(w, TINY, toks)
    for P in (0, 4, 14):
        got = mo.forward_window(w, TINY, toks[:P], toks[P:], list(range(P, 15)))
        np.testing.assert_allclose(got, ref[P:], atol=1e-10, rtol=0)


def test_reordered_window_rows_of_observed_tokens_match_their_logical_forward():
    """Observed tokens moved to the physical prefix keep exactly the logits they have in logical order
    as long as everything before them (logically) is observed too: here the leading run."""
    w = make_model(TINY)
    rng = np.random.default_rng(1)
    toks = rng.integers(0, TINY.vocab - 1, size=12).tolist()
    P = 6
    window = toks[P:]                       # logical slots 0..5; slots 0,1,3 observed
    filled = [1, 1, 0, 1, 0, 0]
    perm = [0, 1, 3, 2, 4, 5]
    phys = [window[j] if filled[j] else TINY.mask_token_id for j in perm]
    got = mo.forward_window(w, TINY, toks[:P], phys, [P + j for j in perm])
    ref = _torch_reference_logits(w, TINY, toks[: P + 2])
    np.testing.assert_allclose(got[:2], ref[P:], atol=1e-10, rtol=0)


def test_loop_with_window_one_is_greedy_decoding_of_the_same_model():
    w = make_model(TINY)
    pt = make_prompts_and_targets(TINY, 1, 6, 8)
    out = mo.decode(w, TINY, pt["prompt"][0], pt["target"][0], tilt=0.0, window=1, max_new_tokens=8,
                    conf_mode="entropy", tau=0.3, lam=0.1, maxprob_thr=0.9)
    seq = pt["prompt"][0].tolist()
    want = []
    for _ in range(8):
        # the logits of a mask token placed at the next position, on top of the text so far
        lg = _torch_reference_logits(w, TINY, seq + [TINY.mask_token_id])[-1]
        tok = int(np.argmax(lg))
        want.append(tok)
        seq.append(tok)
    assert out["y"] == want
