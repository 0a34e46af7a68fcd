"""CUDA path vs the CPU checker, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2202_07471_b200 as sq
from paper_2202_07471_b200 import workloads as W

from cases import SWEEP_SHAPES, adversarial_layer, coarse, redo_layer

pytestmark = pytest.mark.gpu

E, EK, EKC = sq.MODE_E, sq.MODE_E | sq.MODE_K, sq.MODE_EKC


def run_gpu(ws, bits, mode, flags=sq.FLAG_NARROW_RANGE):
    """Quantize a list of numpy layers in one grouped launch; returns LayerBuffers on the host."""
    bufs = [sq.alloc_outputs(torch.from_numpy(np.ascontiguousarray(w)).cuda()) for w in ws]
    for b in bufs:   # poison the outputs so that an unwritten element cannot pass
        b.codes.fill_(-128); b.scales.fill_(float("nan")); b.kernel_err.fill_(float("nan")); b.channel_err.fill_(float("nan"))
    sq.squant_quantize_model(bufs, bits=bits, mode=mode, flags=flags)
    sq.squant_device_status()      # synchronises; raises if a kernel gave up a bounded wait
    return bufs


def assert_layer_equal(b, w, bits, mode, flags=oracle.FLAG_NARROW_RANGE, tag=""):
    r = oracle.quantize_layer(w, bits=bits, mode=mode, flags=flags)
    codes = b.codes.cpu().numpy()
    bad = np.argwhere(codes != r.codes)
    assert bad.size == 0, f"{tag}: {len(bad)} codes differ, first at {bad[0].tolist()}"
    # bit-exact floats: compare the raw words
    assert np.array_equal(b.scales.cpu().numpy().view(np.uint32), r.scales.view(np.uint32)), f"{tag}: scales"
    assert np.array_equal(b.kernel_err.cpu().numpy().view(np.uint32), r.kernel_err.view(np.uint32)), f"{tag}: kernel_err"
    assert np.array_equal(b.channel_err.cpu().numpy().view(np.uint32), r.channel_err.view(np.uint32)), f"{tag}: channel_err"


def test_single_conv_config():
    """Config 1: one [64,64,3,3] layer, N(0, sqrt(2/576)), seed 0, 4 bit, E+K+C."""
    w = W.layer_weights(W.WORKLOADS["single_conv"], 0, seed=0)
    for mode in (E, EK, EKC):
        (b,) = run_gpu([w], 4, mode)
        assert_layer_equal(b, w, 4, mode, tag=f"mode{mode}")


@pytest.mark.parametrize("bits", [2, 3, 4, 6, 8])
def test_shape_sweep_grouped(bits):
    """Every sweep shape in ONE grouped launch: ragged tails, every kernel size path, all group
    sizes, special channels (zero, constant, tiny, huge, ties)."""
    ws = [adversarial_layer(s, seed=17 * bits + i) for i, s in enumerate(SWEEP_SHAPES)]
    for mode in (EKC, EK, E, sq.MODE_E | sq.MODE_C):
        bufs = run_gpu(ws, bits, mode)
        for i, (b, w) in enumerate(zip(bufs, ws)):
            assert_layer_equal(b, w, bits, mode, tag=f"shape{SWEEP_SHAPES[i]} mode{mode}")


def test_e_c_mode_without_k():
    """The E&C ablation (Table 5 of the paper): every element is its own SQuant-C candidate."""
    ws = [adversarial_layer(s, seed=5) for s in [(7, 300, 1, 1), (4, 2049, 1, 1), (6, 64, 3, 3), (3, 2048, 3, 3),
                                                 (5, 7, 5, 5), (9, 1, 3, 3), (4, 3, 7, 7), (3, 33, 2, 2)]]
    mode = sq.MODE_E | sq.MODE_C
    bufs = run_gpu(ws, 4, mode)
    for b, w in zip(bufs, ws):
        assert_layer_equal(b, w, 4, mode)


def test_wide_range_flag():
    w = adversarial_layer((16, 40, 3, 3), seed=2)
    (b,) = run_gpu([w], 4, EKC, flags=0)
    assert_layer_equal(b, w, 4, EKC, flags=0)


def test_unaligned_views_and_null_optional_outputs():
    """Weights and codes that start off a 16-byte boundary take the scalar load/store path."""
    w = adversarial_layer((6, 37, 3, 3), seed=8)
    n = w.size
    base = torch.zeros(n + 3, dtype=torch.float32, device="cuda")
    cbase = torch.full((n + 5,), -128, dtype=torch.int8, device="cuda")
    wv = base[3:3 + n].view(w.shape)
    wv.copy_(torch.from_numpy(w))
    b = sq.LayerBuffers(wv, cbase[5:5 + n].view(w.shape), torch.empty(6, device="cuda"), None, None)
    sq.squant_quantize_model([b], bits=4)
    torch.cuda.synchronize()
    r = oracle.quantize_layer(w, bits=4)
    assert np.array_equal(b.codes.cpu().numpy(), r.codes)
    assert np.array_equal(b.scales.cpu().numpy(), r.scales)
    assert int(cbase[:5].max()) == -128


def test_coarse_grid_ties_large_channel():
    """Heavy ties in both selections on a full-width channel (radix select must fall through
    to the index digits)."""
    w = coarse(W.random_layer((3, 2048, 3, 3), seed=1), steps=24, div=4)
    (b,) = run_gpu([w], 4, EKC)
    assert_layer_equal(b, w, 4, EKC)
    w = np.full((2, 1500, 3, 3), 0.3, dtype=np.float32)
    w[:, 0, 0, 0] = 1.0
    (b,) = run_gpu([w], 8, EKC)
    assert_layer_equal(b, w, 8, EKC)


@pytest.mark.parametrize("bits", [4, 8])
def test_kernels_the_fast_selection_hands_back(bits):
    """3x3 channels in which none, a few, just under half, just over half and all kernels cannot
    be settled by the straight-line selection (tiny weights, error sums near 4): the exact redo
    by list and by per-thread marks."""
    ws = [redo_layer(2048, bits), redo_layer(64, bits, seed=4), redo_layer(8, bits, seed=5)]
    for mode in (EKC, EK):
        bufs = run_gpu(ws, bits, mode)
        for i, (b, w) in enumerate(zip(bufs, ws)):
            assert_layer_equal(b, w, bits, mode, tag=f"redo layer {i} mode{mode}")


@pytest.mark.parametrize("bits,mode", [(4, EKC), (8, EKC), (3, EK)])
def test_long_3x3_channels_pipelined_kernel(bits, mode):
    """Layers of long 3x3 channels (more than 8192 weights each) take the streaming kernel (int8 codes only;
    the pipelined kernel when packed or dequantized outputs are wanted, see the tests of those): several
    such layers of different widths in one launch (one, a few and many more channels than the GPU
    has multiprocessors), next to layers that stay with the grouped kernel, with special channels
    (zero, single non-zero, constant, scales far outside the reciprocal's range, ties)."""
    shapes = [(1, 2048, 3, 3), (5, 1024, 3, 3), (333, 1000, 3, 3), (7, 1400, 3, 3), (40, 2048, 3, 3),
              (9, 912, 3, 3), (6, 2044, 3, 3), (3, 2052, 3, 3), (4, 512, 3, 3), (11, 4100, 1, 1)]
    ws = [adversarial_layer(s, seed=100 * bits + i) for i, s in enumerate(shapes)]
    bufs = run_gpu(ws, bits, mode)
    for i, (b, w) in enumerate(zip(bufs, ws)):
        assert_layer_equal(b, w, bits, mode, tag=f"shape{shapes[i]} mode{mode}")
    # the same buffers again: the work counter of the launch plan starts clean every time
    for b in bufs:
        b.codes.fill_(-128)
    sq.squant_quantize_model(bufs, bits=bits, mode=mode)
    sq.squant_device_status()
    for i, (b, w) in enumerate(zip(bufs, ws)):
        assert_layer_equal(b, w, bits, mode, tag=f"second run shape{shapes[i]}")


def test_random_mixed_launches():
    """Seeded random models mixing long 3x3 layers (streaming kernel), short 3x3, 1x1 and odd kernel
    shapes, random bit widths and modes, each launched twice into the same buffers."""
    rng = np.random.default_rng(12345)
    for trial in range(12):
        shapes = []
        for _ in range(int(rng.integers(1, 7))):
            kind = rng.integers(0, 4)
            if kind == 0:
                shapes.append((int(rng.integers(1, 400)), int(rng.integers(228, 513)) * 4, 3, 3))
            elif kind == 1:
                shapes.append((int(rng.integers(1, 40)), int(rng.integers(1, 228)) * 4, 3, 3))
            elif kind == 2:
                shapes.append((int(rng.integers(1, 60)), int(rng.integers(1, 3000)), 1, 1))
            else:
                shapes.append((int(rng.integers(1, 20)), int(rng.integers(1, 300)), int(rng.integers(1, 6)), int(rng.integers(1, 6))))
        bits = int(rng.choice([2, 3, 4, 6, 8]))
        mode = int(rng.choice([EKC, EK, EKC, EKC]))
        ws = [adversarial_layer(s, seed=7000 + 10 * trial + i) for i, s in enumerate(shapes)]
        bufs = run_gpu(ws, bits, mode)
        for rep in range(2):
            if rep:
                for b in bufs:
                    b.codes.fill_(-128)
                sq.squant_quantize_model(bufs, bits=bits, mode=mode)
                sq.squant_device_status()
            for i, (b, w) in enumerate(zip(bufs, ws)):
                assert_layer_equal(b, w, bits, mode, tag=f"trial {trial} run {rep} shape{shapes[i]} bits{bits} mode{mode}")


@pytest.mark.parametrize("name,bits", [("resnet18", 4), ("resnet50", 4), ("resnet50", 6), ("mobilenetv2", 4),
                                       ("mixed_kernels", 4)])
def test_model_configs_full(name, bits):
    """Configs 2-4 at full size, the whole model in one grouped launch, every element compared."""
    wl = W.WORKLOADS[name]
    ws = [W.layer_weights(wl, i, seed=0, threads=8) for i in range(len(wl.shapes))]
    bufs = run_gpu(ws, bits, EKC)
    for i, (b, w) in enumerate(zip(bufs, ws)):
        assert_layer_equal(b, w, bits, EKC, tag=f"{name} layer {i} {wl.shapes[i]}")


def test_large_layer_config_sampled():
    """Config 5 at full size (8 x [2048,2048,3,3]) in the launch configuration the benchmark
    times; the checker recomputes a sample of whole output channels (channels are independent
    sub-problems), and properties that hold at any size are checked on everything."""
    wl = W.WORKLOADS["large_layer"]
    host = [torch.empty(s, dtype=torch.float32).pin_memory() for s in wl.shapes]
    for i, t in enumerate(host):
        W.layer_weights(wl, i, seed=0, threads=8, out=t.numpy())
    bufs = [sq.alloc_outputs(t.cuda()) for t in host]
    sq.squant_quantize_model(bufs, bits=4, mode=EKC)
    torch.cuda.synchronize()
    for i, b in enumerate(bufs):
        assert int(b.codes.abs().max()) <= 7
        assert float(b.channel_err.abs().max()) <= 0.5          # Eq. 11
        assert float(b.kernel_err.abs().max()) <= 1.0           # r_k = 1.0 after SQuant-C
        tot = b.kernel_err.double().sum(1)
        assert float((tot - b.channel_err.double()).abs().max()) < 1e-3
        pick = np.arange(i, 2048, 61)
        w = host[i].numpy()[pick]
        r = oracle.quantize_layer(w, bits=4, mode=EKC)
        assert np.array_equal(b.codes[pick].cpu().numpy(), r.codes), f"layer {i}"
        assert np.array_equal(b.scales[pick].cpu().numpy(), r.scales)
        assert np.array_equal(b.kernel_err[pick].cpu().numpy(), r.kernel_err)
        assert np.array_equal(b.channel_err[pick].cpu().numpy(), r.channel_err)


def test_host_entry_point_matches_device_entry_point():
    wl = W.WORKLOADS["single_conv"]
    w = W.layer_weights(wl, 0)
    hb = sq.alloc_outputs(torch.from_numpy(w).pin_memory(), pin=True)
    sq.squant_quantize_model_host([hb], bits=4)
    r = oracle.quantize_layer(w, bits=4)
    assert np.array_equal(hb.codes.numpy(), r.codes) and np.array_equal(hb.scales.numpy(), r.scales)
    assert np.array_equal(hb.kernel_err.numpy(), r.kernel_err)
    assert np.array_equal(hb.channel_err.numpy(), r.channel_err)


def test_repeat_calls_are_deterministic_and_counted():
    w = torch.from_numpy(W.random_layer((32, 64, 3, 3), 3)).cuda()
    n0 = sq.squant_launch_count()
    a = sq.squant_quantize_layer(w, bits=4)
    b = sq.squant_quantize_layer(w, bits=4)
    torch.cuda.synchronize()
    assert sq.squant_launch_count() == n0 + 2
    assert torch.equal(a.codes, b.codes) and torch.equal(a.kernel_err, b.kernel_err)


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_reciprocal_division_is_exact_for_every_weight(bits):
    """SQuant-E divides by the channel scale in IEEE fp32 (Algorithm 1, 'Scale and SQuant-E').
    The 3x3 path replaces the division by a per-channel reciprocal plus two fused corrections;
    this runs ALL fp32 weights a channel with the given scale can hold through both and wants
    identical codes and perturbations.  Scales: random ones over the fast range, its two ends,
    powers of two, all-ones significands (worst case for reciprocals)."""
    rng = np.random.default_rng(bits)
    sc = np.exp2(rng.uniform(-60, 60, size=20)).astype(np.float32)
    special = np.array([2.0 ** -60, 2.0 ** 60, 1.0, 3.0, 1.0 / 3.0, 0.007, 5.9604645e-08], dtype=np.float32)
    ones = np.array([0x3f7fffff, 0x3fffffff, 0x2b7fffff, 0x5d7fffff, 0x3f800001, 0x3fc00001], dtype=np.uint32).view(np.float32)
    bad = sq.squant_selfcheck_division(np.concatenate([sc, special, ones]), bits=bits)
    assert not bad.any(), bad


def test_more_layers_than_one_launch_table_holds():
    """More than 96 layers are issued as several launches; results do not depend on the split."""
    shapes = [(3 + (i % 5), 8 + 4 * (i % 7), 3, 3) if i % 3 else (5, 16 + 4 * (i % 9), 1, 1) for i in range(205)]
    ws = [W.random_layer(s, seed=1000 + i) for i, s in enumerate(shapes)]
    n0 = sq.squant_launch_count()
    bufs = run_gpu(ws, 4, EKC)
    assert sq.squant_launch_count() == n0 + 3
    for i, (b, w) in enumerate(zip(bufs, ws)):
        assert_layer_equal(b, w, 4, EKC, tag=f"layer {i} {shapes[i]}")


def test_more_long_channel_layers_than_one_launch_table_holds():
    """The same for the streaming kernel: 101 layers of long 3x3 channels, two launches."""
    shapes = [(1 + (i % 3), 912 + 4 * (i % 11), 3, 3) for i in range(101)]
    ws = [W.random_layer(s, seed=3000 + i) for i, s in enumerate(shapes)]
    n0 = sq.squant_launch_count()
    bufs = run_gpu(ws, 4, EKC)
    assert sq.squant_launch_count() == n0 + 2
    for i, (b, w) in enumerate(zip(bufs, ws)):
        assert_layer_equal(b, w, 4, EKC, tag=f"layer {i} {shapes[i]}")


def test_non_finite_inputs_do_not_disturb_other_channels():
    """NaN / Inf weights are outside the method's domain; their channels produce unspecified
    codes, but every index the kernel forms stays in bounds and finite channels are unaffected."""
    for shape in [(8, 64, 3, 3), (8, 256, 1, 1), (8, 10, 5, 5), (8, 2048, 3, 3), (8, 1000, 3, 3), (300, 1024, 3, 3)]:
        w = W.random_layer(shape, seed=77)
        bad = w.copy()
        bad[1].reshape(-1)[3] = np.nan
        bad[2].reshape(-1)[5] = np.inf
        bad[3].reshape(-1)[::7] = -np.inf
        bad[5].reshape(-1)[:] = np.nan
        (b,) = run_gpu([bad], 4, EKC)
        r = oracle.quantize_layer(w, bits=4, mode=EKC)
        for c in (0, 4, *range(6, shape[0])):
            assert np.array_equal(b.codes[c].cpu().numpy(), r.codes[c])
            assert b.scales[c].item() == r.scales[c]


@pytest.mark.parametrize("bits", [3, 4])
def test_packed_int4_output(bits):
    """SQUANT_FLAG_PACK_INT4: nibble pairs, rows of ceil(NK/2) bytes; all kernel paths, odd and
    even row lengths, bulk-store and plain-store rows."""
    shapes = [(6, 64, 3, 3), (3, 2048, 3, 3), (5, 256, 1, 1), (7, 33, 1, 1), (4, 3, 5, 5), (9, 1, 3, 3), (3, 7, 3, 3)]
    ws = [adversarial_layer(s, seed=3 * bits + i) for i, s in enumerate(shapes)]
    flags = sq.FLAG_NARROW_RANGE | sq.FLAG_PACK_INT4
    bufs = [sq.alloc_outputs(torch.from_numpy(w).cuda(), pack_int4=True) for w in ws]
    for b in bufs:
        b.codes.fill_(-128)
    sq.squant_quantize_model(bufs, bits=bits, mode=EKC, flags=flags)
    sq.squant_device_status()
    for b, w, shp in zip(bufs, ws, shapes):
        r = oracle.quantize_layer(w, bits=bits, mode=EKC, flags=flags)
        assert np.array_equal(b.codes.cpu().numpy(), r.codes), f"shape {shp}"
        assert np.array_equal(b.scales.cpu().numpy(), r.scales)
        assert np.array_equal(b.kernel_err.cpu().numpy(), r.kernel_err)
    with pytest.raises(sq.SquantError):
        sq.squant_quantize_model(bufs[:1], bits=8, flags=flags)


@pytest.mark.parametrize("k", [1, 9])
def test_boundary_bin_between_list_and_radix_capacity(k):
    """SQuant-C boundary bins of every size class: taken whole, ranked from the short list
    (<= 128 members), and the radix-select fallback (129..256 and thousands of tied members)."""
    for members in (40, 128, 129, 200, 256, 257, 700):
        n = 1024
        w = np.zeros((2, n, k), dtype=np.float32)
        w[:, 0, 0] = 127.0                         # scale 1 with bits = 8
        w[:, 1:51, 0] = 0.45                       # 50 candidates at -0.45: taken whole
        w[:, 51:51 + members, 0] = 0.30            # `members` tied candidates at -0.30: boundary bin
        w[1] = -w[1]
        (b,) = run_gpu([w.reshape(2, n, 3, 3) if k == 9 else w.reshape(2, n, 1, 1)], 8, EKC)
        assert_layer_equal(b, w.reshape(2, n, 3, 3) if k == 9 else w.reshape(2, n, 1, 1), 8, EKC, tag=f"members {members}")


def test_dequantized_output():
    """Optional outputs code * s (what Algorithm 1 returns) in fp32 and bfloat16, all paths - the
    pipelined kernel for the long 3x3 channels included -, aligned and not, with int8 and packed codes."""
    shapes = [(6, 64, 3, 3), (3, 2048, 3, 3), (150, 1000, 3, 3), (5, 256, 1, 1), (7, 33, 1, 1), (4, 3, 5, 5), (3, 7, 3, 3)]
    ws = [adversarial_layer(s, seed=40 + i) for i, s in enumerate(shapes)]
    for flags, pack in ((sq.FLAG_NARROW_RANGE, False), (sq.FLAG_NARROW_RANGE | sq.FLAG_PACK_INT4, True)):
        bufs = [sq.alloc_outputs(torch.from_numpy(w).cuda(), dequant=True, pack_int4=pack, dequant_bf16=True) for w in ws]
        for b in bufs:
            b.dequant.fill_(float("nan"))
            b.dequant_bf16.fill_(float("nan"))
        sq.squant_quantize_model(bufs, bits=4, mode=EKC, flags=flags)
        sq.squant_device_status()
        for b, w, shp in zip(bufs, ws, shapes):
            r = oracle.quantize_layer(w, bits=4, mode=EKC, flags=flags, details=True)
            assert np.array_equal(b.dequant.cpu().numpy().view(np.uint32), r.dequant.view(np.uint32)), f"shape {shp}"
            assert np.array_equal(b.dequant_bf16.view(torch.int16).cpu().numpy().view(np.uint16), r.dequant_bf16), f"shape {shp}"
            assert np.array_equal(b.codes.cpu().numpy(), r.codes), f"shape {shp}"
            assert np.array_equal(b.kernel_err.cpu().numpy().view(np.uint32), r.kernel_err.view(np.uint32))
    # bfloat16 alone, on a view that starts off an 8-byte boundary
    w = ws[0]
    base = torch.zeros(w.size + 1, dtype=torch.bfloat16, device="cuda")
    b = sq.alloc_outputs(torch.from_numpy(w).cuda())
    b.dequant_bf16 = base[1:].view(w.shape)
    sq.squant_quantize_model([b], bits=4)
    sq.squant_device_status()
    r = oracle.quantize_layer(w, bits=4, details=True)
    assert np.array_equal(b.dequant_bf16.contiguous().view(torch.int16).cpu().numpy().view(np.uint16), r.dequant_bf16)


def test_host_entry_point_several_chunks_against_the_checker():
    """squant_quantize_model_host takes the layers in chunks of about 64 MB of weights whose
    uploads, launches and downloads overlap on three streams.  Four layers of 75 MB (streaming
    kernel), a small one and a 1x1 one give five chunks; every output is compared with the checker
    on a sample of whole channels of every layer, called twice (cached staging and plans)."""
    shapes = [(512, 2048, 3, 3)] * 4 + [(40, 64, 3, 3), (300, 1000, 1, 1)]
    ws = [W.random_layer(s, seed=900 + i) for i, s in enumerate(shapes)]
    hb = [sq.alloc_outputs(torch.from_numpy(w).pin_memory(), pin=True) for w in ws]
    for rep in range(2):
        for b in hb:
            b.codes.fill_(-128); b.scales.fill_(float("nan")); b.kernel_err.fill_(float("nan")); b.channel_err.fill_(float("nan"))
        sq.squant_quantize_model_host(hb, bits=4)
        sq.squant_device_status()
        for i, (b, w) in enumerate(zip(hb, ws)):
            pick = np.arange(0, w.shape[0], 7) if w.shape[0] > 100 else np.arange(w.shape[0])
            r = oracle.quantize_layer(w[pick], bits=4)
            assert np.array_equal(b.codes.numpy()[pick], r.codes), f"rep {rep} layer {i}"
            assert np.array_equal(b.scales.numpy()[pick].view(np.uint32), r.scales.view(np.uint32))
            assert np.array_equal(b.kernel_err.numpy()[pick].view(np.uint32), r.kernel_err.view(np.uint32))
            assert np.array_equal(b.channel_err.numpy()[pick].view(np.uint32), r.channel_err.view(np.uint32))
            assert int(b.codes.min()) >= -7 and not torch.isnan(b.scales).any()   # every channel was written


def test_one_call_three_kernels():
    """One call whose layers go to three kernels: long 3x3 channels with plain codes (streaming kernel), long 3x3
    channels with a dequantized output (pipelined kernel), short layers (grouped kernel); three launches per
    call, every output compared with the checker, repeated (cached plans, work counters, scratch area)."""
    shapes = [(300, 1024, 3, 3), (200, 2048, 3, 3), (64, 64, 3, 3), (100, 512, 1, 1), (37, 1400, 3, 3)]
    ws = [adversarial_layer(s, seed=31 + i) for i, s in enumerate(shapes)]
    for bits in (4, 8):
        bufs = [sq.alloc_outputs(torch.from_numpy(w).cuda(), dequant=(i in (1, 4)), dequant_bf16=(i == 4)) for i, w in enumerate(ws)]
        count0 = sq.squant_launch_count()
        for rep in range(3):
            for b in bufs:
                b.codes.fill_(-128)
            sq.squant_quantize_model(bufs, bits=bits, mode=EKC)
            sq.squant_device_status()
            for shp, w, b in zip(shapes, ws, bufs):
                assert_layer_equal(b, w, bits, EKC, tag=f"{shp} bits {bits} rep {rep}")
                if b.dequant is not None:
                    r = oracle.quantize_layer(w, bits=bits, mode=EKC)
                    want = r.codes.astype(np.float32) * r.scales.reshape(-1, 1, 1, 1)
                    assert np.array_equal(b.dequant.cpu().numpy().view(np.uint32), want.view(np.uint32)), f"{shp}: dequant"
        assert sq.squant_launch_count() - count0 == 9


@pytest.mark.parametrize("n", [2048, 1500, 1028])
def test_streaming_kernel_hundreds_of_channel_flips(n):
    """Long 3x3 channels whose kernel sums all lean the same way: SQuant-C flips hundreds of kernels per
    channel, with candidates spread over many histogram bins - far more threads are concerned than the
    streaming kernel's queue holds (the rest do their own flips), and the boundary bin is ranked from the
    list.  Weights sit on the 4-bit grid of scale 1/8 except one element per kernel, which is off the grid
    by 0.25 .. 0.49 of a step (downwards in the odd channels)."""
    rng = np.random.default_rng(n)
    m = 6
    w = rng.integers(-6, 7, size=(m, n, 9)).astype(np.float32) * 0.125
    off = rng.uniform(0.25, 0.49, size=(m, n)).astype(np.float32) * 0.125
    sign = np.where(np.arange(m) % 2 == 0, 1.0, -1.0).astype(np.float32)[:, None]
    pos = rng.integers(0, 9, size=(m, n))
    off_grid = rng.integers(-5, 6, size=(m, n)).astype(np.float32) * 0.125 + sign * off
    np.put_along_axis(w, pos[:, :, None], off_grid[:, :, None], axis=2)
    w[:, 0, 0] = 0.875   # absmax: scale 1/8 at 4 bit
    w = w.reshape(m, n, 3, 3)
    (b,) = run_gpu([w], 4, EKC)
    assert_layer_equal(b, w, 4, EKC, tag=f"n {n}")
    r = oracle.quantize_layer(w, bits=4, mode=EKC)
    flips = int(np.abs(np.rint((oracle.quantize_layer(w, bits=4, mode=EK).kernel_err.astype(np.float64).sum(axis=1)))).min())
    assert flips > 200, flips   # the case really has hundreds of flips per channel
    assert np.all(np.abs(r.channel_err) <= 0.5)


@pytest.mark.parametrize("bits,flags", [(2, sq.FLAG_NARROW_RANGE), (6, sq.FLAG_NARROW_RANGE), (4, 0), (8, 0)])
def test_pipelined_kernel_optional_outputs_and_ranges(bits, flags):
    """Long 3x3 channels (streaming kernel) without the optional outputs, at 2 and 6 bit, and
    without the narrow-range flag; one table holds a layer with fewer channels than the GPU has
    multiprocessors and one with many more."""
    shapes = [(9, 1024, 3, 3), (700, 912, 3, 3), (33, 2048, 3, 3)]
    ws = [adversarial_layer(s, seed=50 * bits + i) for i, s in enumerate(shapes)]
    for variant in range(3):   # all outputs, no kernel sums, no sums at all
        bufs = [sq.alloc_outputs(torch.from_numpy(w).cuda(), kernel_err=variant == 0, channel_err=variant <= 1) for w in ws]
        for b in bufs:
            b.codes.fill_(-128)
        sq.squant_quantize_model(bufs, bits=bits, mode=EKC, flags=flags)
        sq.squant_device_status()
        for b, w, shp in zip(bufs, ws, shapes):
            r = oracle.quantize_layer(w, bits=bits, mode=EKC, flags=flags)
            assert np.array_equal(b.codes.cpu().numpy(), r.codes), f"{shp} variant {variant}"
            assert np.array_equal(b.scales.cpu().numpy().view(np.uint32), r.scales.view(np.uint32))
            if b.kernel_err is not None:
                assert np.array_equal(b.kernel_err.cpu().numpy().view(np.uint32), r.kernel_err.view(np.uint32))
            if b.channel_err is not None:
                assert np.array_equal(b.channel_err.cpu().numpy().view(np.uint32), r.channel_err.view(np.uint32))


def test_overlapping_calls_with_different_descriptors():
    """Calls with different descriptors may overlap on the GPU: two models (both with layers for
    the streaming kernel, each with its own work counter and scratch area) on two streams, several rounds."""
    wa = [W.random_layer((200, 1024, 3, 3), seed=61), W.random_layer((50, 64, 3, 3), seed=62)]
    wb = [W.random_layer((300, 912, 3, 3), seed=63), W.random_layer((64, 300, 1, 1), seed=64)]
    ba = [sq.alloc_outputs(torch.from_numpy(w).cuda()) for w in wa]
    bb = [sq.alloc_outputs(torch.from_numpy(w).cuda()) for w in wb]
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(5):
        sq.squant_quantize_model(ba, bits=4, stream=s1)
        sq.squant_quantize_model(bb, bits=4, stream=s2)
    sq.squant_device_status()
    for bufs, ws in ((ba, wa), (bb, wb)):
        for b, w in zip(bufs, ws):
            assert_layer_equal(b, w, 4, EKC)


def _clip_scales(w, bits, lo=1.5, hi=4.0, seed=0):
    """Per-channel scales 1.5 to 4 times smaller than the absmax scale (so that elements clip), with a
    few special ones: the absmax scale itself, a far too large one, and invalid ones (-> 1)."""
    m = w.shape[0]
    qmax = 2 ** (bits - 1) - 1
    a = np.abs(w.reshape(m, -1)).max(1)
    a[a == 0] = 1.0
    rng = np.random.default_rng(seed)
    sc = (a / qmax / rng.uniform(lo, hi, size=m)).astype(np.float32)
    sc[::5] = (a[::5] / np.float32(qmax)).astype(np.float32)
    if m > 3:
        sc[3] = np.float32(a[3] * 50)
    if m > 7:
        sc[6] = 0.0
        sc[7] = np.nan
    return sc


@pytest.mark.parametrize("bits,flags", [(4, sq.FLAG_NARROW_RANGE), (3, 0), (8, sq.FLAG_NARROW_RANGE)])
def test_caller_supplied_scales(bits, flags):
    """Algorithm 1 with its scale as an input: the clip of Sec. 2.2 fires, clipped elements are
    never flipped outward and kernels / channels can run out of candidates.  All kernel sizes, long
    3x3 channels included (they leave the persistent kernels), modes E, E|K, E|K|C and E|C on 1x1."""
    shapes = [(12, 64, 3, 3), (9, 7, 3, 3), (10, 300, 1, 1), (6, 2049, 1, 1), (8, 5, 5, 5), (16, 1, 3, 3), (5, 3, 7, 7),
              (4, 1024, 3, 3), (3, 33, 2, 2)]
    ws = [W.random_layer(s, seed=300 + i) for i, s in enumerate(shapes)]
    scs = [_clip_scales(w, bits, seed=i) for i, w in enumerate(ws)]
    for mode in (EKC, EK, E):
        bufs = [sq.alloc_outputs(torch.from_numpy(w).cuda()) for w in ws]
        for b, sc in zip(bufs, scs):
            b.scales_in = torch.from_numpy(sc).cuda()
            b.codes.fill_(-128)
        sq.squant_quantize_model(bufs, bits=bits, mode=mode, flags=flags)
        sq.squant_device_status()
        for b, w, sc, shp in zip(bufs, ws, scs, shapes):
            r = oracle.quantize_layer(w, bits=bits, mode=mode, flags=flags, scales_in=sc)
            assert np.array_equal(b.codes.cpu().numpy(), r.codes), f"{shp} mode {mode}"
            assert np.array_equal(b.scales.cpu().numpy().view(np.uint32), r.scales.view(np.uint32))
            assert np.array_equal(b.kernel_err.cpu().numpy().view(np.uint32), r.kernel_err.view(np.uint32)), f"{shp} mode {mode}"
            assert np.array_equal(b.channel_err.cpu().numpy().view(np.uint32), r.channel_err.view(np.uint32)), f"{shp} mode {mode}"
    # E|C: 1x1 layers only
    mode = sq.MODE_E | sq.MODE_C
    bufs = [sq.alloc_outputs(torch.from_numpy(ws[i]).cuda()) for i in (2, 3)]
    for b, i in zip(bufs, (2, 3)):
        b.scales_in = torch.from_numpy(scs[i]).cuda()
    sq.squant_quantize_model(bufs, bits=bits, mode=mode, flags=flags)
    sq.squant_device_status()
    for b, i in zip(bufs, (2, 3)):
        r = oracle.quantize_layer(ws[i], bits=bits, mode=mode, flags=flags, scales_in=scs[i])
        assert np.array_equal(b.codes.cpu().numpy(), r.codes) and np.array_equal(b.channel_err.cpu().numpy(), r.channel_err)
    b = sq.alloc_outputs(torch.from_numpy(ws[0]).cuda())
    b.scales_in = torch.from_numpy(scs[0]).cuda()
    with pytest.raises(sq.SquantError):
        sq.squant_quantize_model([b], bits=bits, mode=mode, flags=flags)


def test_caller_supplied_scales_other_outputs_and_host_path():
    """Supplied scales with packed int4 and dequantized outputs, and through the host-buffer call."""
    shapes = [(6, 64, 3, 3), (5, 256, 1, 1), (4, 3, 5, 5)]
    ws = [W.random_layer(s, seed=340 + i) for i, s in enumerate(shapes)]
    scs = [_clip_scales(w, 4, seed=20 + i) for i, w in enumerate(ws)]
    flags = sq.FLAG_NARROW_RANGE | sq.FLAG_PACK_INT4
    bufs = [sq.alloc_outputs(torch.from_numpy(w).cuda(), dequant=True, pack_int4=True) for w in ws]
    for b, sc in zip(bufs, scs):
        b.scales_in = torch.from_numpy(sc).cuda()
    sq.squant_quantize_model(bufs, bits=4, flags=flags)
    sq.squant_device_status()
    for b, w, sc in zip(bufs, ws, scs):
        r = oracle.quantize_layer(w, bits=4, flags=flags, scales_in=sc, details=True)
        assert np.array_equal(b.codes.cpu().numpy(), r.codes)
        assert np.array_equal(b.dequant.cpu().numpy().view(np.uint32), r.dequant.view(np.uint32))
    hb = [sq.alloc_outputs(torch.from_numpy(w).pin_memory(), pin=True) for w in ws]
    for b, sc in zip(hb, scs):
        b.scales_in = torch.from_numpy(sc).pin_memory()
    sq.squant_quantize_model_host(hb, bits=4)
    for b, w, sc in zip(hb, ws, scs):
        r = oracle.quantize_layer(w, bits=4, scales_in=sc)
        assert np.array_equal(b.codes.numpy(), r.codes) and np.array_equal(b.kernel_err.numpy(), r.kernel_err)
        assert np.array_equal(b.scales.numpy(), r.scales)


def test_failure_path_status_word_and_expiring_wait():
    """Every wait inside the kernels is bounded; one that runs out sets a device status word that
    squant_device_status reports once (SQUANT_ERR_TIMEOUT) and clears.  The plumbing is exercised
    without disturbing any solver launch: by writing the word from the host, and by a one-warp
    kernel whose wait on a barrier nobody arrives at runs out after 64 polls and returns.  The
    context stays usable: a normal call afterwards matches the checker."""
    sq.squant_device_status()                          # clean to start with
    sq.squant_debug_set_status(1)
    with pytest.raises(sq.SquantError) as ei:
        sq.squant_device_status()
    assert ei.value.code == -10
    sq.squant_device_status()                          # reported once, then cleared
    sq.squant_debug_wait_expires(64)
    with pytest.raises(sq.SquantError) as ei:
        sq.squant_device_status()
    assert ei.value.code == -10
    sq.squant_device_status()
    w = W.random_layer((40, 1024, 3, 3), seed=12)      # streaming kernel: its work counters were reset with the status
    (b,) = run_gpu([w], 4, EKC)
    assert_layer_equal(b, w, 4, EKC)


def _edge_scale_case(n):
    """One channel of n 1x1 kernels in which the absmax element lands a shade above qmax (its flip
    would leave the range) and every other element ties with it in perturbation: SQuant-C must
    skip the edge element although it comes first in the tie order."""
    qmax = np.float32(127.0)
    a = None
    for t in np.linspace(1.0, 2.0, 4000, dtype=np.float32):
        if np.float32(t) / (np.float32(t) / qmax) > qmax:
            a = np.float32(t)
            break
    assert a is not None
    s = a / qmax
    w = np.full((1, n, 1, 1), s * np.float32(2.0 ** -17), dtype=np.float32)
    w[0, 0, 0, 0] = a
    return w


def test_channels_wider_than_one_thread_block():
    """Channels that do not fit one thread block's shared memory take the cluster kernel (2 to 8
    blocks per output channel, absmax / channel sum / select histograms exchanged through
    distributed shared memory).  Fully connected layers of 100,000 and 262,143 inputs, 3x3 and 5x5
    layers with 8192 and 2600 kernels per channel, every mode, special channels; and the case in
    which the range exclusion binds (70,000 tied candidates, the first of them on the clip edge)."""
    shapes = [(3, 100000, 1, 1), (2, 8192, 3, 3), (2, 2600, 5, 5), (2, 262143, 1, 1), (9, 46001, 1, 1), (3, 4100, 3, 3)]
    ws = [adversarial_layer(s, seed=500 + i) for i, s in enumerate(shapes)]
    n0 = sq.squant_launch_count()
    for bits, mode in ((4, EKC), (8, EK), (3, E)):
        bufs = run_gpu(ws, bits, mode)
        for b, w, shp in zip(bufs, ws, shapes):
            assert_layer_equal(b, w, bits, mode, tag=f"{shp} bits {bits} mode {mode}")
    assert sq.squant_launch_count() == n0 + 3 * (4 + 1)   # one cluster launch per wide layer; the last two shapes still fit one block
    w = _edge_scale_case(70000)
    for mode in (EKC, sq.MODE_E | sq.MODE_C):
        (b,) = run_gpu([w], 8, mode)
        r = oracle.quantize_layer(w, bits=8, mode=mode, details=True)
        assert r.codes[0, 0, 0, 0] == 127 and r.codes[0, 1, 0, 0] == 1 and int(r.codes[0, 2:].max()) == 0   # the checker skipped the edge element
        assert_layer_equal(b, w, 8, mode, tag=f"edge case mode {mode}")
    # a wide layer next to ordinary ones in one call; packed and dequantized outputs; supplied scales
    ws2 = [W.random_layer((4, 64, 3, 3), seed=1), W.random_layer((2, 70001, 1, 1), seed=2), W.random_layer((3, 9000, 3, 3), seed=3)]
    flags = sq.FLAG_NARROW_RANGE | sq.FLAG_PACK_INT4
    bufs = [sq.alloc_outputs(torch.from_numpy(w).cuda(), pack_int4=True, dequant=True, dequant_bf16=True) for w in ws2]
    scs = [None, _clip_scales(ws2[1], 4, seed=1), _clip_scales(ws2[2], 4, seed=2)]
    for b, sc in zip(bufs, scs):
        b.codes.fill_(-128)
        if sc is not None:
            b.scales_in = torch.from_numpy(sc).cuda()
    sq.squant_quantize_model(bufs, bits=4, flags=flags)
    sq.squant_device_status()
    for b, w, sc in zip(bufs, ws2, scs):
        r = oracle.quantize_layer(w, bits=4, flags=flags, details=True, scales_in=sc)
        assert np.array_equal(b.codes.cpu().numpy(), r.codes), w.shape
        assert np.array_equal(b.kernel_err.cpu().numpy().view(np.uint32), r.kernel_err.view(np.uint32)), w.shape
        assert np.array_equal(b.channel_err.cpu().numpy().view(np.uint32), r.channel_err.view(np.uint32))
        assert np.array_equal(b.dequant.cpu().numpy().view(np.uint32), r.dequant.view(np.uint32))
        assert np.array_equal(b.dequant_bf16.view(torch.int16).cpu().numpy().view(np.uint16), r.dequant_bf16)
    with pytest.raises(sq.SquantError):   # beyond the select key's 18 index bits
        sq.squant_plan_info([(1, 262144, 1, 1)])


def test_checked_build_finds_no_violation_on_small_cases():
    """The checked build of the library (every shared-memory / table index verified, each 3x3
    channel's error sum taken a second time from its final codes by plain division) runs the
    sweep of small shapes, the 3x3 cases the fast selection hands back, long 3x3 channels through the
    streaming kernel, and a cluster case: no check fails, and its results are the regular build's."""
    from paper_2202_07471_b200 import build as lib_build
    import os
    if not os.path.exists(lib_build.LIB_DEBUG):
        pytest.skip("libsquant_debug.so has not been built")
    ws = [adversarial_layer(s, seed=9 + i) for i, s in enumerate(SWEEP_SHAPES)] + [redo_layer(64, 4, seed=4), redo_layer(2048, 4)]
    # long 3x3 channels (streaming kernel): special channels, heavy ties (digit-by-digit selection), a partial last warp
    ws += [adversarial_layer((150, 1000, 3, 3), seed=77), coarse(W.random_layer((5, 2048, 3, 3), seed=78), steps=24, div=4)]
    ref = run_gpu(ws, 4, EKC)
    sq.use_library(lib_build.LIB_DEBUG)
    try:
        checked, n, site = sq.squant_debug_violations()
        assert checked and n == 0
        for mode in (EKC, EK, sq.MODE_E | sq.MODE_C):
            bufs = run_gpu(ws, 4, mode)
            _, n, site = sq.squant_debug_violations()
            assert n == 0, f"{n} failed checks, first at site {site}, mode {mode}"
            if mode == EKC:
                for a, b in zip(bufs, ref):
                    assert torch.equal(a.codes, b.codes) and torch.equal(a.kernel_err.view(torch.int32), b.kernel_err.view(torch.int32))
        (b,) = run_gpu([W.random_layer((2, 70001, 1, 1), seed=2)], 4, EKC)
        assert sq.squant_debug_violations()[1] == 0
    finally:
        sq.use_library(None)
    assert sq.squant_debug_violations()[0] is False      # the regular build has no checks
