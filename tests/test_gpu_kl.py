"""Parity of dmr_stepwise_kl (through the C ABI) with the fp64 oracle on the same seeded logits.

Tolerance: fp32 with ex2.approx (2 ulp) and log2 (1 ulp): the three terms S1/S0, lse(a), lse(b) are each
accurate to a few 1e-7 relative and lse is of order 10, so |KL_gpu - KL_ref| <= 5e-6 + 1e-4 KL_ref.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2602_02711_b200 as dmr
from paper_2602_02711_b200 import inputs
from helpers import to_dev_bf16

pytestmark = pytest.mark.gpu

ABS, REL = 5e-6, 1e-4


def close(got, want):
    got = np.asarray(got, dtype=np.float64)
    return np.all(np.abs(got - want) <= ABS + REL * np.abs(want))


def run_case(T, V, dtype, seed, mean_len=12):
    high, low = inputs.logit_pair(T, V, seed=seed, index=V)
    offs = inputs.step_offsets(T, mean_len, seed=seed, index=T)
    if dtype == "bf16":
        hb, lb = inputs.f64_to_bf16_bits(high), inputs.f64_to_bf16_bits(low)
        want_s, want_t = oracle.stepwise_kl(hb, lb, offs)
        hd, ld = to_dev_bf16(hb), to_dev_bf16(lb)
    else:
        h32, l32 = high.astype(np.float32), low.astype(np.float32)
        want_s, want_t = oracle.stepwise_kl(h32, l32, offs)
        hd, ld = torch.from_numpy(h32).cuda(), torch.from_numpy(l32).cuda()
    od = torch.from_numpy(offs).cuda()
    ks, kt = dmr.dmr_stepwise_kl(hd, ld, od)
    assert close(kt.cpu().numpy(), want_t)
    assert close(ks.cpu().numpy(), want_s)
    # deterministic, and independent of how many tokens share the launch
    ks2, kt2 = dmr.dmr_stepwise_kl(hd, ld, od)
    assert torch.equal(kt, kt2) and torch.equal(ks, ks2)
    if T > 3:
        _, kt3 = dmr.dmr_stepwise_kl(hd[1:4].clone(), ld[1:4].clone(), torch.tensor([0, 3], dtype=torch.int32).cuda())
        assert torch.equal(kt3, kt[1:4])
    return kt


@pytest.mark.parametrize("T,V,dtype", [
    (37, 1000, "bf16"),      # V a multiple of 8, ragged against the 512 x 16-thread stride
    (5, 151936, "bf16"),     # a full vocabulary: 37 vector iterations per thread and a tail
    (9, 1003, "bf16"),       # V not a multiple of 8: element-wise path
    (21, 4096, "f32"),
    (4, 1001, "f32"),
    (1, 8, "bf16"),          # fewer entries than threads
    (1500, 512, "bf16"),     # more tokens than resident CTAs: grid-stride over tokens
])
def test_stepwise_kl_matches_oracle(T, V, dtype):
    run_case(T, V, dtype, seed=11)


def test_identical_logits_give_exactly_zero():
    high, _ = inputs.logit_pair(7, 2048, seed=2)
    hd = to_dev_bf16(inputs.f64_to_bf16_bits(high))
    ks, kt = dmr.dmr_stepwise_kl(hd, hd.clone(), torch.tensor([0, 7], dtype=torch.int32).cuda())
    assert torch.all(kt == 0) and torch.all(ks == 0)


def test_large_logits_and_zero_probability_entries():
    high, low = inputs.logit_pair(6, 640, seed=3)
    high[:, 5] += 300.0          # far beyond e^88: only the running maximum keeps this finite
    low[:, 5] += 280.0
    high[:, 9] = -np.inf         # probability 0 under the high-precision model
    low[:, 9] = -np.inf
    low[:, 11] = -1.0e4
    h32, l32 = high.astype(np.float32), low.astype(np.float32)
    want_s, want_t = oracle.stepwise_kl(h32, l32, [0, 6])
    ks, kt = dmr.dmr_stepwise_kl(torch.from_numpy(h32).cuda(), torch.from_numpy(l32).cuda(),
                                 torch.tensor([0, 6], dtype=torch.int32).cuda())
    assert np.all(np.isfinite(kt.cpu().numpy()))
    assert close(kt.cpu().numpy(), want_t) and close(ks.cpu().numpy(), want_s)


def test_empty_steps_and_no_tokens():
    high, low = inputs.logit_pair(4, 256, seed=4)
    hd, ld = to_dev_bf16(inputs.f64_to_bf16_bits(high)), to_dev_bf16(inputs.f64_to_bf16_bits(low))
    offs = torch.tensor([0, 0, 2, 2, 4, 4], dtype=torch.int32).cuda()
    ks, kt = dmr.dmr_stepwise_kl(hd, ld, offs)
    k = kt.cpu().numpy().astype(np.float64)
    want = np.array([0.0, np.float32(np.float32(k[0]) + np.float32(k[1])) / 2, 0.0, np.float32(np.float32(k[2]) + np.float32(k[3])) / 2, 0.0])
    assert np.allclose(ks.cpu().numpy(), want, rtol=1e-6, atol=0)
    ks0, kt0 = dmr.dmr_stepwise_kl(hd[:0], ld[:0], torch.tensor([0, 0], dtype=torch.int32).cuda())
    assert kt0.numel() == 0 and ks0.cpu().tolist() == [0.0]


def test_argument_errors():
    a = torch.zeros((2, 16), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(dmr.DmrError):
        dmr.dmr_stepwise_kl(a, torch.zeros((2, 16), dtype=torch.float32, device="cuda"), torch.tensor([0, 2], dtype=torch.int32).cuda())
    with pytest.raises(dmr.DmrError):
        dmr.dmr_stepwise_kl(a, torch.zeros((3, 16), dtype=torch.bfloat16, device="cuda"), torch.tensor([0, 2], dtype=torch.int32).cuda())
