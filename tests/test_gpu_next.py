"""GPU parity of the later-stage entry points against the oracle, through the C ABI: block-prefix gate
(Algorithm 1, Step 1), threshold equation, accepted-prefix length (Algorithm 1, Step 4)."""
import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2512_08537_b200 as ardiff
from gpu_util import dev_bf16, require_cuda

pytestmark = pytest.mark.gpu
ENT_TOL = 1e-3
BAND = 1e-4


def check_blocks(bits, r, gamma, tau):
    Hs, mask_o, idx_o, count_o, len_o = oracle.gate_blocks(bits, r, gamma, tau)
    mask, idx, count, blen, row_ent, tok_ent = ardiff.ardiff_entropy_gate_blocks(dev_bf16(bits), r, gamma, tau,
                                                                                 want_token_entropy=True)
    torch.cuda.synchronize()
    n = len(Hs)
    mask_g, c = mask.cpu().numpy(), int(count.item())
    idx_g, len_g, ent_g = idx.cpu().numpy()[:c], blen.cpu().numpy(), tok_ent.cpu().numpy()[:n]
    nan = np.isnan(Hs)
    assert np.array_equal(np.isnan(ent_g), nan)
    assert np.all(np.abs(ent_g[~nan] - Hs[~nan]) <= ENT_TOL)
    # self-consistency (bit-exact): idx = ascending positions of the mask, lengths = per-block sums, mask is a
    # prefix inside every block
    assert c == int(mask_g.sum()) and np.array_equal(idx_g, np.flatnonzero(mask_g).astype(np.int32))
    nb = (n + gamma - 1) // gamma
    pad = np.zeros(nb * gamma, np.uint8)
    pad[:n] = mask_g
    blocks = pad.reshape(nb, gamma)
    assert np.array_equal(len_g, blocks.sum(axis=1).astype(np.int32))
    assert np.all(np.diff(blocks.astype(np.int8), axis=1) <= 0)
    # against the oracle: exact for every block none of whose tokens sits in the band around tau
    in_band = np.zeros(nb * gamma, bool)
    in_band[:n] = ~nan & (np.abs(Hs - float(np.float32(tau))) < BAND)
    clean = ~in_band.reshape(nb, gamma).any(axis=1)
    pad_o = np.zeros(nb * gamma, np.uint8)
    pad_o[:n] = mask_o
    assert np.array_equal(blocks[clean], pad_o.reshape(nb, gamma)[clean])
    assert np.array_equal(len_g[clean], len_o[clean])
    if clean.all():
        assert c == count_o and np.array_equal(idx_g, idx_o)
    return c


@pytest.mark.parametrize("gamma", [1, 2, 8, 37, 4096])
@pytest.mark.parametrize("n", [1, 63, 1000, 4099])
def test_block_prefix_gate_single_row_tokens(n, gamma):
    wl = synth.workload("cfg2", n=n)
    bits = synth.features(wl)
    H = oracle.entropy(bits)
    tau = float(np.quantile(H, 0.15)) if n > 1 else float(H[0]) - 0.5
    check_blocks(bits, 1, gamma, tau)


@pytest.mark.parametrize("r,d", [(4, 256), (16, 64), (3, 1001)])
def test_block_prefix_gate_mean_over_rows(r, d):
    wl = synth.workload("cfg1", n=515 * r, d=d)
    bits = synth.features(wl)
    Hs = oracle.entropy(bits).reshape(-1, r).mean(axis=1)
    check_blocks(bits, r, 8, float(np.quantile(Hs, 0.1)))


def test_block_prefix_gate_workload_cfg2_blocks_of_8():
    wl = synth.workload("cfg2")
    bits = synth.features(wl)
    H = oracle.entropy(bits)
    kept = check_blocks(bits, 1, 8, float(np.quantile(H, 0.05)))
    assert 0 < kept < wl.n


def test_block_gate_with_gamma_one_equals_plain_gate_and_empty_input():
    dev = require_cuda()
    wl = synth.workload("cfg1", n=777)
    feat = dev_bf16(synth.features(wl))
    _, _, _, ent = ardiff.ardiff_entropy_gate(feat, -1.0, want_entropy=True)
    tau = float(ent.median().item())
    mask_a, idx_a, count_a, _ = ardiff.ardiff_entropy_gate(feat, tau)
    mask_b, idx_b, count_b, blen, _, _ = ardiff.ardiff_entropy_gate_blocks(feat, 1, 1, tau)
    torch.cuda.synchronize()
    c = int(count_a.item())
    assert c == int(count_b.item()) and torch.equal(mask_a, mask_b) and torch.equal(idx_a[:c], idx_b[:c])
    assert torch.equal(blen, mask_a.to(torch.int32))
    empty = torch.empty((0, 64), dtype=torch.bfloat16, device=dev)
    _, _, count0, _, _, _ = ardiff.ardiff_entropy_gate_blocks(empty, 1, 8, 0.0)
    assert int(count0.item()) == 0


@pytest.mark.parametrize("n", [1, 7, 1024, 100003])
def test_tau_calibration(n):
    dev = require_cuda()
    rng = np.random.default_rng(n)
    H = rng.uniform(0.2, 7.0, size=n).astype(np.float32)
    got = ardiff.ardiff_tau_calibrate(torch.from_numpy(H).to(dev)).cpu().numpy()
    m, s, t = oracle.tau_calibrate(H.astype(np.float64))
    assert abs(got[0] - m) <= 1e-12 * max(1.0, abs(m)) + 1e-13
    assert abs(got[1] - s) <= 1e-10 and abs(got[2] - t) <= 1e-10
    again = ardiff.ardiff_tau_calibrate(torch.from_numpy(H).to(dev)).cpu().numpy()
    assert np.array_equal(got, again)                                 # fixed summation order


def test_tau_calibration_from_the_gates_own_entropies():
    wl = synth.workload("cfg2")
    bits = synth.features(wl)
    _, _, _, ent = ardiff.ardiff_entropy_gate(dev_bf16(bits), -1.0, want_entropy=True)
    got = ardiff.ardiff_tau_calibrate(ent).cpu().numpy()
    m, s, t = oracle.tau_calibrate(oracle.entropy(bits))
    assert abs(got[0] - m) <= 1e-3 and abs(got[1] - s) <= 1e-3 and abs(got[2] - t) <= 4e-4


@pytest.mark.parametrize("gamma", [1, 4, 8, 37, 5000])
def test_accept_prefix(gamma):
    dev = require_cuda()
    rng = np.random.default_rng(gamma)
    n = 4099
    r = rng.uniform(0, 1, n).astype(np.float32)
    ratio = rng.uniform(0.5, 2.0, n).astype(np.float32)
    ratio[::97] = r[::97]                                              # ties are not rejections
    got = ardiff.ardiff_accept_prefix(torch.from_numpy(r).to(dev), torch.from_numpy(ratio).to(dev), gamma)
    assert np.array_equal(got.cpu().numpy(), oracle.accept_prefix(r, ratio, gamma))


@pytest.mark.parametrize("gamma", [1, 8, 37])
def test_accept_prefix_on_truncated_blocks(gamma):
    """Algorithm 1 Step 4 on the draft that Step 1 left: the accepted count is capped by the kept length."""
    dev = require_cuda()
    rng = np.random.default_rng(50 + gamma)
    n = 4099
    nb = (n + gamma - 1) // gamma
    r = rng.uniform(0, 1, n).astype(np.float32)
    ratio = rng.uniform(0.5, 2.0, n).astype(np.float32)
    full = np.array([min(gamma, n - b * gamma) for b in range(nb)], np.int32)
    kept = np.minimum(rng.integers(0, gamma + 1, nb).astype(np.int32), full)
    got = ardiff.ardiff_accept_prefix(torch.from_numpy(r).to(dev), torch.from_numpy(ratio).to(dev), gamma,
                                      block_len=torch.from_numpy(kept).to(dev))
    assert np.array_equal(got.cpu().numpy(), oracle.accept_prefix(r, ratio, gamma, kept))


def test_early_stop_feeds_accept_prefix_on_the_device():
    """Step 1 -> Step 4 composed on the device: block_len written by the block-prefix gate is read by the
    accepted-prefix kernel on the same stream, no host round trip."""
    dev = require_cuda()
    wl = synth.workload("cfg2", n=8 * 515)
    bits = synth.features(wl)
    H = oracle.entropy(bits)
    tau = float(np.quantile(H, 0.1))
    rng = np.random.default_rng(9)
    r = rng.uniform(0, 1, wl.n).astype(np.float32)
    ratio = rng.uniform(0.7, 2.0, wl.n).astype(np.float32)
    _, _, _, blen, _, _ = ardiff.ardiff_entropy_gate_blocks(dev_bf16(bits), 1, 8, tau)
    got = ardiff.ardiff_accept_prefix(torch.from_numpy(r).to(dev), torch.from_numpy(ratio).to(dev), 8, block_len=blen)
    _, _, _, _, len_o = oracle.gate_blocks(bits, 1, 8, tau)
    band = (np.abs(H - float(np.float32(tau))) < BAND).reshape(-1, 8).any(axis=1)
    want = oracle.accept_prefix(r, ratio, 8, len_o)
    assert np.array_equal(got.cpu().numpy()[~band], want[~band])
    assert np.all(got.cpu().numpy() <= blen.cpu().numpy())


def test_block_prefix_gate_without_row_entropy_output_and_on_the_two_pass_shape():
    """The one-pass kernel keeps row entropies in shared memory (the caller need not take them); a draft
    block whose rows exceed a CTA's shared memory goes through the row-entropy array instead and needs it."""
    dev = require_cuda()
    wl = synth.workload("cfg2", n=3000)
    bits = synth.features(wl)
    feat = dev_bf16(bits)
    H = oracle.entropy(bits)
    tau = float(np.quantile(H, 0.1))
    a = ardiff.ardiff_entropy_gate_blocks(feat, 1, 8, tau, want_token_entropy=True)
    b = ardiff.ardiff_entropy_gate_blocks(feat, 1, 8, tau, want_token_entropy=True, want_row_entropy=False)
    torch.cuda.synchronize()
    assert b[4] is None and torch.equal(a[0], b[0]) and torch.equal(a[3], b[3]) and torch.equal(a[5], b[5])
    assert int(a[2].item()) == int(b[2].item())
    # 30000 single-row tokens per draft block: beyond the one-pass limit
    wl2 = synth.workload("cfg1", n=70001, d=64)
    bits2 = synth.features(wl2)
    tau2 = float(np.quantile(oracle.entropy(bits2), 0.0005))
    check_blocks(bits2, 1, 30000, tau2)
    with pytest.raises(ardiff.ArdiffError):
        ardiff.ardiff_entropy_gate_blocks(dev_bf16(bits2), 1, 30000, tau2, want_row_entropy=False)


@pytest.mark.parametrize("name,n,d", [("cfg2", 16384, 768), ("cfg4", 5000, 5120), ("cfg1", 77, 12)])
def test_gate_with_threshold_statistics_in_one_pass(name, n, d):
    """ardiff_entropy_gate_stats: the gate's usual outputs plus mean / std / tau of its own entropies."""
    require_cuda()
    wl = synth.workload(name, n=n, d=d)
    bits = synth.features(wl)
    feat = dev_bf16(bits)
    H = oracle.entropy(bits)
    tau = float(np.quantile(H, 0.3))
    mask, idx, count, ent, out3 = ardiff.ardiff_entropy_gate_stats(feat, tau, want_entropy=True)
    mask_p, idx_p, count_p, ent_p = ardiff.ardiff_entropy_gate(feat, tau, want_entropy=True)
    torch.cuda.synchronize()
    c = int(count.item())
    assert c == int(count_p.item()) and torch.equal(mask, mask_p) and torch.equal(idx[:c], idx_p[:c])
    assert torch.equal(ent, ent_p)
    got = out3.cpu().numpy()
    m, s, t = oracle.tau_calibrate(H)
    assert abs(got[0] - m) <= 1e-3 and abs(got[1] - s) <= 1e-3 and abs(got[2] - t) <= 4e-4
    # against the two-pass fp64 kernel on the very same fp32 entropies: only the summation order differs
    ref = ardiff.ardiff_tau_calibrate(ent).cpu().numpy()
    assert np.all(np.abs(got - ref) <= 1e-11)
    again = ardiff.ardiff_entropy_gate_stats(feat, tau)[4].cpu().numpy()
    assert np.array_equal(got, again)                                  # fixed merge order
