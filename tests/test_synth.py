"""The seeded input generators: layouts of the paper's model families and counter-based values."""
import math

import numpy as np
import pytest
import torch

from paper_2012_05396_b200 import synth


def test_layout_sizes():
    # parameter counts of the standard architectures (trainable tensors, no conv biases in ResNets)
    expect = {"resnet20": (59, 269722), "resnet56": (167, 853018),
              "resnet50": (161, 25557032), "vgg16": (32, 138357544)}
    for name, (T, N) in expect.items():
        lay = synth.get_layout(name)
        assert (lay.num_tensors, lay.numel) == (T, N)
        offs = lay.offsets
        assert all(o % synth.ALIGN_ELEMS == 0 for o in offs)
        assert all(offs[t] + lay.numels[t] <= offs[t + 1] for t in range(T - 1))
        assert offs[-1] + lay.numels[-1] <= lay.padded_numel < N + synth.ALIGN_ELEMS * T
    assert max(synth.get_layout("vgg16").numels) == 25088 * 4096
    assert synth.get_layout("resnet50").numels[0] == 64 * 3 * 7 * 7


def test_generators_are_deterministic_and_element_addressable():
    lay = synth.get_layout("resnet20")
    g = synth.gradient(lay, 3, 1, 1e-2)
    assert torch.equal(g, synth.gradient(lay, 3, 1, 1e-2))
    assert not torch.equal(g, synth.gradient(lay, 3, 2, 1e-2))
    assert not torch.equal(g, synth.gradient(lay, 4, 1, 1e-2))
    idx = torch.tensor([0, 1, 431, 432, 435, 269721, 269723], dtype=torch.int64)
    assert torch.equal(g[idx], synth.gradient_at(lay, 3, 1, 1e-2, idx))
    # alignment padding carries zero gradient and zero weight
    mask = synth.valid_mask(lay)
    assert int(mask.sum()) == lay.numel
    assert float(g[mask == 0].abs().max()) == 0.0
    assert float(synth.init_weights(lay)[mask == 0].abs().max()) == 0.0


def test_distributions():
    n = 1 << 20
    x = synth.normal(synth.stream_key(synth.SEED, synth.STREAM_GRAD, 0, 0), n, 1e-3)
    assert abs(float(x.mean())) < 5e-6 and abs(float(x.std()) / 1e-3 - 1) < 5e-3
    u = synth.uniform_buffer(synth.STREAM_GRAD, n)
    assert -1.0 <= float(u.min()) and float(u.max()) < 1.0
    assert abs(float(u.mean())) < 3e-3 and abs(float(u.std()) - 1 / math.sqrt(3)) < 3e-3
    lay = synth.get_layout("resnet20")
    w = synth.init_weights(lay)
    t = lay.names.index("s1.b0.conv1.weight")
    off, cnt = lay.offsets[t], lay.numels[t]
    assert abs(float(w[off:off + cnt].std()) / math.sqrt(2.0 / (16 * 9)) - 1) < 0.05
    t = lay.names.index("stem.bn.gamma")
    assert torch.all(w[lay.offsets[t]:lay.offsets[t] + 16] == 1.0)


def test_mixer_matches_splitmix64_reference_values():
    # First outputs of SplitMix64 seeded with 0 (the published generator: state += golden; mix(state)).
    golden = 0x9E3779B97F4A7C15
    outs = [synth._mix_int(golden * i) for i in (1, 2, 3)]
    assert outs == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    t = torch.tensor([synth._s64(golden * i) for i in (1, 2, 3)], dtype=torch.int64)
    got = [int(v) & ((1 << 64) - 1) for v in synth._mix_tensor(t)]
    assert got == outs


def test_bf16_bits_roundtrip():
    x = synth.uniform_buffer(synth.STREAM_GRAD, 1000)
    b = synth.to_bf16(x)
    bits = synth.bf16_bits(b)
    back = torch.from_numpy((bits.astype(np.uint32) << 16).view(np.float32).copy())
    assert torch.equal(back, b.to(torch.float32))


@pytest.mark.gpu
def test_cpu_and_cuda_generate_identical_bytes():
    lay = synth.get_layout("resnet56")
    for it, wk in ((0, 0), (7, 3)):
        a = synth.gradient(lay, it, wk, 1e-2, device="cpu")
        b = synth.gradient(lay, it, wk, 1e-2, device="cuda")
        assert torch.equal(a, b.cpu())
    assert torch.equal(synth.init_weights(lay, device="cpu"), synth.init_weights(lay, device="cuda").cpu())
    assert torch.equal(synth.uniform_buffer(synth.STREAM_PRE, 100003, device="cpu"),
                       synth.uniform_buffer(synth.STREAM_PRE, 100003, device="cuda").cpu())
