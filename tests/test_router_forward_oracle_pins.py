"""Pins of the oracle's router forward pass (Sec. 4.1 "Router Architecture": X_t + P_t through a masked Transformer
encoder, last-valid-step pooling, Softmax(W h*)).

The paper fixes no width, normalisation placement or activation; the reading taken (post-layer-norm encoder layer, ReLU,
key-padding mask, eps = 1e-5) is the one of the standard library encoder layer, so that layer - a different code base -
pins the oracle; invariants that hold for any correct encoder pin what a library call cannot: padded steps never matter,
without positional embeddings the earlier steps may be permuted, a one-step sequence needs no attention at all.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_02711_b200 import inputs

CFG = dict(d=64, heads=4, ffn=128, layers=3, l_max=12, classes=3)


def torch_reference(Z, lengths, p, heads):
    d = Z.shape[2]
    ffn = p["layers"][0]["w1"].shape[0]
    layer = torch.nn.TransformerEncoderLayer(d_model=d, nhead=heads, dim_feedforward=ffn, dropout=0.0, activation="relu",
                                             batch_first=True, norm_first=False, dtype=torch.float64)
    enc = torch.nn.TransformerEncoder(layer, num_layers=len(p["layers"]), enable_nested_tensor=False)
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    with torch.no_grad():
        for mod, lay in zip(enc.layers, p["layers"]):
            mod.self_attn.in_proj_weight.copy_(t(lay["wqkv"]))
            mod.self_attn.in_proj_bias.copy_(t(lay["bqkv"]))
            mod.self_attn.out_proj.weight.copy_(t(lay["wo"]))
            mod.self_attn.out_proj.bias.copy_(t(lay["bo"]))
            mod.linear1.weight.copy_(t(lay["w1"]))
            mod.linear1.bias.copy_(t(lay["b1"]))
            mod.linear2.weight.copy_(t(lay["w2"]))
            mod.linear2.bias.copy_(t(lay["b2"]))
            mod.norm1.weight.copy_(t(lay["ln1_g"]))
            mod.norm1.bias.copy_(t(lay["ln1_b"]))
            mod.norm2.weight.copy_(t(lay["ln2_g"]))
            mod.norm2.bias.copy_(t(lay["ln2_b"]))
        enc.eval()
        B, L, _ = Z.shape
        x = t(Z) + t(p["pos"])[:L][None]
        pad = torch.arange(L)[None, :] >= torch.from_numpy(np.asarray(lengths, dtype=np.int64))[:, None]
        H = enc(x, src_key_padding_mask=pad)
        hstar = H[torch.arange(B), torch.from_numpy(np.asarray(lengths, dtype=np.int64)) - 1]
        logits = hstar @ t(p["wc"]).T + t(p["bc"])
        return torch.softmax(logits, dim=-1).numpy()


def test_matches_the_library_encoder_layer():
    p = inputs.router_params(**CFG, seed=1)
    B, L = 6, 9
    Z = inputs.router_embeddings(B, L, CFG["d"], seed=1)
    n = inputs.router_lengths(B, L, seed=1)
    got = oracle.router_forward(Z, n, p, CFG["heads"])
    want = torch_reference(Z, n, p, CFG["heads"])
    assert got.shape == (B, CFG["classes"])
    assert np.abs(got - want).max() <= 1e-12
    assert np.abs(got.sum(axis=1) - 1.0).max() <= 1e-14


def test_padded_steps_never_matter():
    p = inputs.router_params(**CFG, seed=2)
    B, L = 4, 10
    Z = inputs.router_embeddings(B, L, CFG["d"], seed=2)
    n = np.array([1, 4, 7, 10], dtype=np.int32)
    base = oracle.router_forward(Z, n, p, CFG["heads"])
    Z2 = Z.copy()
    for b in range(B):
        Z2[b, n[b]:, :] = 1e3 * (b + 1)            # garbage behind the valid steps
    assert np.array_equal(oracle.router_forward(Z2, n, p, CFG["heads"]), base)
    for b in range(B):                             # the same sequence alone, without padding
        alone = oracle.router_forward(Z[b:b + 1, :n[b]], n[b:b + 1], p, CFG["heads"])
        assert np.abs(alone[0] - base[b]).max() <= 1e-13


def test_without_positions_earlier_steps_may_be_permuted():
    # attention over the valid steps is a set operation; only the last step is singled out (it is the one pooled)
    p = inputs.router_params(**CFG, seed=3)
    p["pos"] = np.zeros_like(p["pos"])
    L = 8
    Z = inputs.router_embeddings(1, L, CFG["d"], seed=3)
    n = np.array([L], dtype=np.int32)
    base = oracle.router_forward(Z, n, p, CFG["heads"])
    perm = np.array([3, 0, 6, 1, 5, 2, 4, 7])
    assert np.abs(oracle.router_forward(Z[:, perm], n, p, CFG["heads"]) - base).max() <= 1e-12
    moved_last = np.array([7, 1, 2, 3, 4, 5, 6, 0])
    assert np.abs(oracle.router_forward(Z[:, moved_last], n, p, CFG["heads"]) - base).max() >= 1e-6
    # with positional embeddings the order matters
    q = inputs.router_params(**CFG, seed=3)
    assert np.abs(oracle.router_forward(Z[:, perm], n, q, CFG["heads"]) - oracle.router_forward(Z, n, q, CFG["heads"])).max() >= 1e-6


def test_one_step_sequence_is_a_plain_mlp():
    # one valid step: the softmax over a single key is 1, so attention returns the value vector whatever q and k are
    p = inputs.router_params(d=16, heads=2, ffn=24, layers=2, l_max=4, classes=2, seed=4)
    Z = inputs.router_embeddings(1, 3, 16, seed=4)
    got = oracle.router_forward(Z, np.array([1], dtype=np.int32), p, 2)[0]

    def ln(x, g, b):
        mu = sum(x) / len(x)
        var = sum((v - mu) ** 2 for v in x) / len(x)
        return [(v - mu) / (var + 1e-5) ** 0.5 * gg + bb for v, gg, bb in zip(x, g, b)]

    def affine(W, bias, x):
        return [sum(float(w) * v for w, v in zip(row, x)) + float(bb) for row, bb in zip(W, bias)]

    d = 16
    x = [float(a) + float(b) for a, b in zip(Z[0, 0], p["pos"][0])]
    for lay in p["layers"]:
        v = affine(lay["wqkv"][2 * d:], lay["bqkv"][2 * d:], x)
        y = affine(lay["wo"], lay["bo"], v)
        x = ln([a + b for a, b in zip(x, y)], [float(t) for t in lay["ln1_g"]], [float(t) for t in lay["ln1_b"]])
        h = [max(t, 0.0) for t in affine(lay["w1"], lay["b1"], x)]
        y = affine(lay["w2"], lay["b2"], h)
        x = ln([a + b for a, b in zip(x, y)], [float(t) for t in lay["ln2_g"]], [float(t) for t in lay["ln2_b"]])
    logits = affine(p["wc"], p["bc"], x)
    m = max(logits)
    e = [np.exp(t - m) for t in logits]
    want = np.array(e) / sum(e)
    assert np.abs(got - want).max() <= 1e-12


def test_rejects_bad_lengths():
    p = inputs.router_params(**CFG, seed=5)
    Z = inputs.router_embeddings(2, 4, CFG["d"], seed=5)
    with pytest.raises(ValueError):
        oracle.router_forward(Z, np.array([0, 2]), p, CFG["heads"])
    with pytest.raises(ValueError):
        oracle.router_forward(Z, np.array([2, 5]), p, CFG["heads"])
