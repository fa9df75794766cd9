"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on
identical seeded inputs.

Bar: packed words and grad_in bit-identical; y within 2 ulp of the storage
dtype of the exactly rounded binary64 value.  Both sides use the SAME table
(read back from the library with fewbit_table_get), so the comparison isolates
the hot path; the solver is compared with the oracle's DP in the CPU tests.
"""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import oracle
import paper_2202_00441_b200 as fb
from paper_2202_00441_b200 import workloads as wl
from helpers import bf16_bits_to_f32, finite_mask, ulp_distance

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
GUARD = 64            # guard elements / words placed around every output buffer
TORCH_DT = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}
_THREADS = max(1, len(os.sched_getaffinity(0)))
_POOL = ThreadPoolExecutor(max_workers=_THREADS)
_TABLES = {}


def table(act, bits):
    key = (act, bits)
    if key not in _TABLES:
        _TABLES[key] = fb.fewbit_table_create(act, bits)
    return _TABLES[key]


def np_bits(t: torch.Tensor) -> np.ndarray:
    return wl.to_numpy_bits(t)


def guarded(n, dtype, fill):
    """A device buffer of n elements with GUARD canary elements on both sides.
    The payload starts 256-byte aligned."""
    pad = 256 // torch.empty(0, dtype=dtype).element_size()
    assert GUARD <= pad
    buf = torch.full((n + 2 * pad,), fill, dtype=dtype, device=DEV)
    return buf, buf[pad:pad + n], pad


def check_guards(buf, n, pad, fill):
    assert bool((buf[:pad] == fill).all()) and bool((buf[pad + n:] == fill).all()), "wrote outside the buffer"


def run_gpu(act, bits, x, g, inplace=False):
    """fwd + bwd through the C ABI with canaries around every output."""
    t = table(act, bits)
    n = x.numel()
    words = fb.fewbit_packed_bytes(n, bits) // 4
    pbuf, packed, ppad = guarded(words, torch.int32, 0x5A5A5A5A)
    if inplace:
        y, gi = x.clone(), g.clone()
        fb.fewbit_fwd(t, y, y, packed)
        fb.fewbit_bwd(t, packed, gi, gi)
    else:
        fill = 777.0
        ybuf, y, ypad = guarded(n, x.dtype, fill)
        gbuf, gi, gpad = guarded(n, x.dtype, fill)
        fb.fewbit_fwd(t, x, y, packed)
        fb.fewbit_bwd(t, packed, g, gi)
        torch.cuda.synchronize()
        check_guards(ybuf, n, ypad, fill)
        check_guards(gbuf, n, gpad, fill)
    torch.cuda.synchronize()
    check_guards(pbuf, words, ppad, 0x5A5A5A5A)
    return y, packed, gi


def _unpack_on_device(pk, bits, n):
    w = pk.view(torch.int32).to(torch.int64) & 0xFFFFFFFF
    pos = torch.arange(n, device=DEV, dtype=torch.int64) * bits
    lo = w[pos >> 5] >> (pos & 31)
    nxt = w[torch.clamp((pos >> 5) + 1, max=w.numel() - 1)] << (32 - (pos & 31))
    return (lo | torch.where((pos & 31) + bits > 32, nxt, torch.zeros_like(lo))) & ((1 << bits) - 1)


def oracle_block(act, bits, s, lev, x_np, g_np):
    y, p = oracle.fwd(act, bits, s, x_np)
    gi = oracle.bwd(bits, lev, p, g_np)
    return y, p, gi


def compare_block(act, bits, x_np, g_np, y_np, p_np, gi_np, what):
    s, lev = table(act, bits).arrays()
    y_ref, p_ref, gi_ref = oracle_block(act, bits, s, lev, x_np, g_np)
    assert np.array_equal(p_np[:p_ref.size], p_ref), f"{what}: packed codes differ"
    raw = np.uint32 if gi_np.dtype == np.float32 else np.uint16
    assert np.array_equal(gi_np.view(raw), gi_ref.view(raw)), f"{what}: grad_in differs"
    ok = finite_mask(x_np)
    d = ulp_distance(y_np[ok], y_ref[ok])
    assert d.size == 0 or d.max() <= 2, f"{what}: y off by {d.max()} ulp"


def compare_full(act, bits, x, g, y, packed, gi, what):
    compare_block(act, bits, np_bits(x), np_bits(g), np_bits(y), np_bits(packed).view(np.uint32), np_bits(gi), what)


def compare_every_element(act, bits, x, g, y, packed, gi, what):
    """compare_full for tensors of any size: the arrays go to the host once and are cut into one
    contiguous shard per host thread (on multiples of 1024 elements, so every shard's packed words are
    whole); every element of y and grad_in and every packed word is compared with the oracle."""
    n = x.numel()
    xn, gn, yn, gin = np_bits(x), np_bits(g), np_bits(y), np_bits(gi)
    pn = np_bits(packed).view(np.uint32)
    shards = max(1, min(4 * _THREADS, n // (1 << 20)))
    jobs = []
    for r in range(shards):
        lo, hi = wl.shard_range(n, r, shards, 1024)
        if hi > lo:
            jobs.append((lo, xn[lo:hi], gn[lo:hi], yn[lo:hi], pn[lo // 32 * bits:(hi * bits + 31) // 32], gin[lo:hi]))
    list(_POOL.map(lambda j: compare_block(act, bits, j[1], j[2], j[3], j[4], j[5], f"{what} @ {j[0]}"), jobs))


def compare_sampled(act, bits, x, g, y, packed, gi, what, blocks=24, block_elems=8192, seed=0, also_at=()):
    """Element-by-element comparison on randomly placed 32-aligned blocks plus
    the first and the last (ragged) block (and blocks starting at `also_at`)."""
    n = x.numel()
    rng = np.random.default_rng(seed)
    starts = {0, max(0, (n - block_elems) // 32 * 32)} | {int(a) // 32 * 32 for a in also_at}
    while len(starts) < blocks:
        starts.add(int(rng.integers(0, max(1, n - block_elems))) // 32 * 32)
    jobs = []
    for e0 in sorted(starts):
        m = min(block_elems, n - e0)
        w0 = e0 // 32 * bits
        w1 = (((e0 + m) * bits) + 31) // 32
        jobs.append((e0, np_bits(x[e0:e0 + m]), np_bits(g[e0:e0 + m]), np_bits(y[e0:e0 + m]),
                     np_bits(packed[w0:w1]).view(np.uint32), np_bits(gi[e0:e0 + m])))
    list(_POOL.map(lambda j: compare_block(act, bits, j[1], j[2], j[3], j[4], j[5], f"{what} @ {j[0]}"), jobs))


# --------------------------------------------------------------------------
# the five configurations
# --------------------------------------------------------------------------
def test_config1_gelu3_f32_full():
    x, g = wl.draw(wl.C1, DEV)
    for act in wl.C1.acts:
        for bits in wl.C1.bits:
            y, p, gi = run_gpu(act, bits, x, g)
            compare_full(act, bits, x, g, y, p, gi, "c1")


def test_config2_silu_bf16_full():
    x, g = wl.draw(wl.C2, DEV)
    for bits in wl.C2.bits:
        y, p, gi = run_gpu("silu", bits, x, g)
        n = x.numel()
        cuts = [wl.shard_range(n, r, 8, 1024) for r in range(8)]
        jobs = []
        for lo, hi in cuts:
            jobs.append(("silu", bits, np_bits(x[lo:hi]), np_bits(g[lo:hi]), np_bits(y[lo:hi]),
                         np_bits(p[lo // 32 * bits:(hi * bits + 31) // 32]).view(np.uint32), np_bits(gi[lo:hi]), f"c2 k={bits}"))
        list(_POOL.map(lambda j: compare_block(*j), jobs))


def test_config3_gelu_bf16_llm_ffn_every_element():
    x, g = wl.draw(wl.C3, DEV)
    assert x.numel() == 2 ** 28
    for bits in wl.C3.bits:
        y, p, gi = run_gpu("gelu", bits, x, g)
        compare_every_element("gelu", bits, x, g, y, p, gi, f"c3 k={bits}")
        # every code of the full-size launch against torch.bucketize, 2^26 elements at a time
        s, _ = table("gelu", bits).arrays()
        edges = torch.tensor(s, device=DEV)
        step = 1 << 26
        for e0 in range(0, x.numel(), step):
            want = torch.bucketize(x[e0:e0 + step].float(), edges, right=False)
            got = _unpack_on_device(p[e0 // 32 * bits:(e0 + step) // 32 * bits], bits, step)
            assert torch.equal(got, want), (bits, e0)
            del want, got
        del y, p, gi


def test_config4_cnn_f32_every_element():
    x, g = wl.draw(wl.C4, DEV)
    for act in wl.C4.acts:
        y, p, gi = run_gpu(act, 2, x, g)
        compare_every_element(act, 2, x, g, y, p, gi, f"c4 {act}")


@pytest.mark.parametrize("n", [2 ** 16, 2 ** 20])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_config5_sweep_small_full(n, dtype):
    case = next(c for c in wl.sweep_cases([n]) if c.dtype == dtype)
    x, g = wl.draw(case, DEV)
    for act in case.acts:
        for bits in case.bits:
            y, p, gi = run_gpu(act, bits, x, g)
            compare_full(act, bits, x, g, y, p, gi, f"c5 {act} k={bits} n={n} {dtype}")


@pytest.mark.parametrize("n", [2 ** 24, 2 ** 24 + 7, 2 ** 28])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_config5_sweep_large_sampled(n, dtype):
    case = next(c for c in wl.sweep_cases([n]) if c.dtype == dtype)
    x, g = wl.draw(case, DEV)
    blocks = 12 if n < 2 ** 28 else 8
    # every element for two activations (the heaviest arithmetic and one with an exponential in both
    # tails), sampled blocks for the others; at 2^24 (+7) every element of all seven
    everywhere = case.acts if n < 2 ** 28 else ("gelu", "softplus")
    for act in case.acts:
        for bits in case.bits:
            y, p, gi = run_gpu(act, bits, x, g)
            what = f"c5 {act} k={bits} n={n} {dtype}"
            if act in everywhere:
                compare_every_element(act, bits, x, g, y, p, gi, what)
            else:
                compare_sampled(act, bits, x, g, y, p, gi, what, blocks=blocks, block_elems=4096, seed=bits)
            del y, p, gi


@pytest.mark.parametrize("act", ["gelu", "tanh", "relu"])
def test_f32_codes_for_every_input_pattern(act, table_mode):
    """All 2^32 binary32 patterns through fewbit_fwd, 256 M at a time: the packed codes equal
    #{j : s_j < x} computed by torch.bucketize on the same inputs (NaN -> 0), for every bucketize
    variant the size-based choice, the forced table and the forced search select."""
    chunk = 1 << 28
    base = torch.arange(chunk, device=DEV, dtype=torch.int64)
    for bits in (2, 3, 4):
        t = table(act, bits)
        s_np, _ = t.arrays()
        bounds = torch.from_numpy(np.ascontiguousarray(s_np)).to(DEV)
        shifts = torch.arange(0, 32, bits, device=DEV, dtype=torch.int64)[: 32 // bits] if 32 % bits == 0 else None
        for c in range(16):
            x = (base + c * chunk).to(torch.int32).view(torch.float32) if c < 8 else \
                (base + c * chunk - (1 << 32)).to(torch.int32).view(torch.float32)
            _, pk = fb.fewbit_fwd(t, x)
            want = torch.bucketize(x, bounds, right=False).to(torch.int64)
            want = torch.where(torch.isnan(x), torch.zeros_like(want), want)
            words = pk.view(torch.int32).to(torch.int64) & 0xFFFFFFFF
            if shifts is not None:                      # 2 and 4 bits: codes do not straddle words
                got = ((words[:, None] >> shifts[None, :]) & ((1 << bits) - 1)).reshape(-1)
            else:                                       # 3 bits: 32 codes in 3 words
                w3 = words.view(-1, 3)
                bitsream = w3[:, 0] | (w3[:, 1] << 32)  # low 64 bits, then the top word
                idx = torch.arange(32, device=DEV, dtype=torch.int64) * 3
                lo = (bitsream[:, None] >> idx[None, :].clamp(max=61)) & 7
                hi_bits = (w3[:, 1] >> 31) | (w3[:, 2] << 1)      # stream bits 63 ..
                hi = (hi_bits[:, None] >> (idx[None, :] - 63).clamp(min=0)) & 7
                got = torch.where(idx[None, :] >= 63, hi, lo).reshape(-1)
            assert torch.equal(got, want), (act, bits, c)
            del x, pk, want, words, got


def test_shards_cut_by_shard_range_concatenate_to_the_single_launch_stream():
    """The multi-GPU path is N independent launches on the ranges `workloads.shard_range` cuts (no
    exchange step).  Here the shards of a 3- and an 8-way split run one after another on one GPU:
    their outputs, concatenated, are the single-launch y, packed stream and grad_in, bit for bit."""
    n = (1 << 22) + 5 * 1024 + 77
    x = torch.randn(n, device=DEV).mul_(1.5).bfloat16()
    g = torch.randn(n, device=DEV).bfloat16()
    for bits in (1, 3, 4):
        t = table("silu", bits)
        y, pk = fb.fewbit_fwd(t, x)
        gi = fb.fewbit_bwd(t, pk, g)
        for world in (3, 8):
            ys, pks, gis = [], [], []
            for rank in range(world):
                lo, hi = wl.shard_range(n, rank, world)
                ysh, psh = fb.fewbit_fwd(t, x[lo:hi])
                gis.append(fb.fewbit_bwd(t, psh, g[lo:hi]))
                ys.append(ysh)
                pks.append(psh)
            torch.cuda.synchronize()
            assert torch.equal(torch.cat(ys).view(torch.int16), y.view(torch.int16))
            assert torch.equal(torch.cat(pks), pk), (bits, world)
            assert torch.equal(torch.cat(gis).view(torch.int16), gi.view(torch.int16))


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_randomised_tables_sizes_dtypes_under_every_variant(seed):
    """Random activation, bit width, dtype, size (ragged, whole warp-blocks, several waves), built-in
    or injected tables (random boundaries, duplicates, tiny and large scales), inputs with zeros,
    infinities, NaNs and subnormals: every bucketize variant (search, table with dynamic and with
    static distribution, size-based choice) gives the same y and packed words, and the codes are
    torch.bucketize's."""
    import random
    rng = random.Random(seed)
    nprng = np.random.default_rng(seed)
    acts = wl.ACTIVATIONS + wl.EXTRA_ACTIVATIONS
    for _ in range(40):
        dtype, act, bits = rng.choice(["f32", "bf16", "f16"]), rng.choice(acts), rng.randint(1, 4)
        n = rng.choice([rng.randint(1, 5000), rng.randint(5000, 3_000_000), 1024 * rng.randint(1, 3000), (1 << 23) + rng.randint(0, 3000)])
        if rng.random() < 0.5:
            t = table(act, bits)
        else:
            s = np.sort(nprng.standard_normal((1 << bits) - 1).astype(np.float32) * np.float32(10.0 ** rng.uniform(-3, 1.5)))
            if bits > 1 and rng.random() < 0.3:
                s[rng.randrange(s.size - 1) + 1] = s[0]
                s = np.sort(s)
            t = fb.fewbit_table_from_arrays(act, bits, s, nprng.standard_normal(1 << bits).astype(np.float32))
        x = (torch.randn(n, device=DEV) * 10.0 ** rng.uniform(-2, 1.3)).to(TORCH_DT[dtype])
        if n > 10:
            special = rng.choice([0.0, -0.0, float("inf"), float("-inf"), float("nan"), 1e-40, -1e-40, 65504.0, -3e38])
            x[torch.randint(0, n, (min(n, 50),), device=DEV)] = torch.tensor(special, device=DEV).to(TORCH_DT[dtype])
        s_np, _ = t.arrays()
        want = torch.bucketize(x.float(), torch.from_numpy(np.ascontiguousarray(s_np)).to(DEV), right=False)
        want = torch.where(torch.isnan(x.float()), torch.zeros_like(want), want)
        outs = []
        for mode, queue in (("never", None), ("always", None), ("always", "never"), ("auto", None)):
            fb.fewbit_set_option("fwd_table", mode)
            if queue:
                fb.fewbit_set_option("fwd_queue", queue)
            else:
                fb.fewbit_set_option("fwd_queue", "auto")
            outs.append(fb.fewbit_fwd(t, x))
        torch.cuda.synchronize()
        what = (seed, dtype, act, bits, n)
        assert torch.equal(_unpack_on_device(outs[0][1], bits, n), want), what
        for y, pk in outs[1:]:
            assert torch.equal(pk, outs[0][1]) and torch.equal(y.view(torch.uint8), outs[0][0].view(torch.uint8)), what


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_degenerate_boundary_tables(dtype):
    """Injected tables at the edges of what Eq. 2 allows: all boundaries equal, infinite boundaries,
    boundaries at the smallest subnormal, at +-0 and beyond the binary16 range; inputs with zeros,
    infinities, NaN, subnormals and the largest finite values.  Codes are torch.bucketize's under
    every bucketize variant."""
    inf = float("inf")
    cases = {1: [[0], [inf], [-inf], [1e-45], [-1e-45], [65520], [3.4e38]],
             2: [[0, 0, 0], [-inf, 0, inf], [-inf, -inf, -inf], [inf, inf, inf], [-3e38, 0, 3e38], [1e-45, 1e-45, 2e-45],
                 [-0.0, 0.0, 0.0], [65504, 65504, 65520]],
             3: [[-inf, -1, -1, 0, 1, 1, inf], [1e30] * 7],
             4: [[-inf] * 5 + [0] * 5 + [inf] * 5, list(np.linspace(-1e-44, 1e-44, 15)), [7] * 15]}
    special = [0.0, -0.0, inf, -inf, float("nan"), 1e-45, -1e-45, 1e-40, -1e-40, 6e-8, -6e-8, 65504.0, -65504.0, 65520.0,
               3.3e38, -3.3e38, 7.0, 1.0, -1.0]
    for bits, tables in cases.items():
        for s in tables:
            t = fb.fewbit_table_from_arrays("tanh", bits, np.array(s, dtype=np.float32), np.arange(1 << bits, dtype=np.float32))
            s_np, _ = t.arrays()
            edges = torch.from_numpy(np.ascontiguousarray(s_np)).to(DEV)
            for n in (70000, (1 << 23) + 5):
                x = (torch.randn(n, device=DEV) * 3).to(TORCH_DT[dtype])
                x[:len(special)] = torch.tensor(special, device=DEV).to(TORCH_DT[dtype])
                want = torch.bucketize(x.float(), edges, right=False)
                want = torch.where(torch.isnan(x.float()), torch.zeros_like(want), want)
                for mode, queue in (("never", None), ("always", None), ("always", "never")):
                    fb.fewbit_set_option("fwd_table", mode)
                    if queue:
                        fb.fewbit_set_option("fwd_queue", queue)
                    else:
                        fb.fewbit_set_option("fwd_queue", "auto")
                    _, pk = fb.fewbit_fwd(t, x)
                    assert torch.equal(_unpack_on_device(pk, bits, n), want), (dtype, bits, s, n, mode, queue)


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_backward_with_special_levels_and_gradients(dtype):
    """Levels and incoming gradients at the edges of the arithmetic (infinities, NaN, signed zeros,
    subnormals, the largest finite values): grad_in is torch's binary32 product rounded once -- the
    same bits wherever that is a number, NaN where it is NaN."""
    inf, nan = float("inf"), float("nan")
    lev = np.array([inf, -inf, nan, 0.0, -0.0, 1e-45, -1e-45, 3e38, -3e38, 1.0, -1.0, 1e-30, 65504.0, 65520.0, 2.0 ** -24, 0.3],
                   dtype=np.float32)
    s = np.linspace(-2, 2, 15).astype(np.float32)
    t = fb.fewbit_table_from_arrays("tanh", 4, s, lev)
    special = torch.tensor([0.0, -0.0, inf, -inf, nan, 1e-45, 1e-40, -1e-40, 65504.0, 3e38, -3e38, 1.0], device=DEV)
    gen = torch.Generator(device=DEV).manual_seed(5)
    for n, scale in ((5000, 1.0), ((1 << 22) + 77, 1e3), (1 << 20, 1e-3)):
        x = (torch.randn(n, generator=gen, device=DEV) * 1.5).to(TORCH_DT[dtype])
        g = (torch.randn(n, generator=gen, device=DEV) * scale).to(TORCH_DT[dtype])
        for at in (0, 100, 300, 1024, n - 12):
            g[at:at + special.numel()] = special.to(TORCH_DT[dtype])
        _, pk = fb.fewbit_fwd(t, x)
        gi = fb.fewbit_bwd(t, pk, g)
        codes = torch.bucketize(x.float(), torch.from_numpy(s).to(DEV), right=False)
        want = (g.float() * torch.from_numpy(lev).to(DEV)[codes]).to(TORCH_DT[dtype])
        assert torch.equal(torch.isnan(gi), torch.isnan(want)), (dtype, n)
        number = ~torch.isnan(want)
        assert torch.equal(gi[number].view(torch.uint8), want[number].view(torch.uint8)), (dtype, n)


@pytest.mark.parametrize("seed", [6, 7])
def test_randomised_folded_tables_under_every_variant(seed):
    """Folded tables (caption of Fig. 3) with random range and grid, random dtype, size and input
    scale: the codes are torch.bucketize's of |x| (NaN -> 0), the same under every bucketize variant,
    and the backward product is torch's binary32 product rounded once."""
    import random
    rng = random.Random(seed)
    for _ in range(30):
        dtype, act, bits = rng.choice(["f32", "bf16", "f16"]), rng.choice(["sigmoid", "tanh"]), rng.randint(1, 4)
        t = fb.fewbit_table_create_folded(act, bits, B=rng.uniform(2.0, 12.0), n_cells=rng.choice([64, 257, 1000, 2048, 4096]))
        n = rng.choice([rng.randint(1, 5000), rng.randint(5000, 3_000_000), 1024 * rng.randint(1, 3000), (1 << 23) + rng.randint(0, 3000)])
        x = (torch.randn(n, device=DEV) * 10.0 ** rng.uniform(-2, 1.3)).to(TORCH_DT[dtype])
        if n > 10:
            special = rng.choice([0.0, -0.0, float("inf"), float("-inf"), float("nan"), 1e-40, -1e-40, 65504.0, -3e38])
            x[torch.randint(0, n, (min(n, 50),), device=DEV)] = torch.tensor(special, device=DEV).to(TORCH_DT[dtype])
        g = torch.randn(n, device=DEV).to(TORCH_DT[dtype])
        s_np, lev = t.arrays()
        want = torch.bucketize(x.float().abs(), torch.from_numpy(np.ascontiguousarray(s_np)).to(DEV), right=False)
        want = torch.where(torch.isnan(x.float()), torch.zeros_like(want), want)
        outs = []
        for mode, queue in (("never", None), ("always", None), ("always", "never"), ("auto", None)):
            fb.fewbit_set_option("fwd_table", mode)
            if queue:
                fb.fewbit_set_option("fwd_queue", queue)
            else:
                fb.fewbit_set_option("fwd_queue", "auto")
            outs.append(fb.fewbit_fwd(t, x))
        torch.cuda.synchronize()
        what = (seed, dtype, act, bits, n)
        assert torch.equal(_unpack_on_device(outs[0][1], bits, n), want), what
        for y, pk in outs[1:]:
            assert torch.equal(pk, outs[0][1]) and torch.equal(y.view(torch.uint8), outs[0][0].view(torch.uint8)), what
        gi = fb.fewbit_bwd(t, outs[0][1], g)
        prod = (g.float() * torch.from_numpy(np.ascontiguousarray(lev)).to(DEV)[want]).to(TORCH_DT[dtype])
        assert torch.equal(gi.view(torch.uint8), prod.view(torch.uint8)), what


@pytest.mark.parametrize("seed", [4, 5])
def test_randomised_backward_and_bias_against_torch_arithmetic(seed):
    """Random sizes, dtypes, activations and bit widths: grad_in equals torch's binary32 product
    rounded once, and f(x + bias) equals the plain forward on torch's binary32 sum rounded once."""
    import random
    rng = random.Random(seed)
    for _ in range(40):
        dtype, act, bits = rng.choice(["f32", "bf16", "f16"]), rng.choice(wl.ACTIVATIONS + wl.EXTRA_ACTIVATIONS), rng.randint(1, 4)
        t = table(act, bits)
        _, lev = t.arrays()
        n = rng.choice([rng.randint(1, 5000), rng.randint(5000, 2_000_000), 1024 * rng.randint(1, 2000)])
        x = (torch.randn(n, device=DEV) * 2).to(TORCH_DT[dtype])
        g = (torch.randn(n, device=DEV) * 10.0 ** rng.uniform(-6, 3)).to(TORCH_DT[dtype])
        _, pk = fb.fewbit_fwd(t, x)
        gi = fb.fewbit_bwd(t, pk, g)
        codes = _unpack_on_device(pk, bits, n)
        want = (g.float() * torch.from_numpy(np.ascontiguousarray(lev)).to(DEV)[codes]).to(TORCH_DT[dtype])
        assert torch.equal(gi.view(torch.uint8), want.view(torch.uint8)), (seed, dtype, act, bits, n)
        cols = 8 * rng.randint(1, 1500)
        rows = rng.randint(1, max(1, 400000 // cols))
        xb = (torch.randn(rows, cols, device=DEV) * 2).to(TORCH_DT[dtype])
        b = torch.randn(cols, device=DEV).to(TORCH_DT[dtype])
        z = (xb.float() + b.float()[None, :]).to(TORCH_DT[dtype])
        for mode in ("never", "always"):
            fb.fewbit_set_option("fwd_table", mode)
            y1, p1 = fb.fewbit_fwd_bias(t, xb, b)
            y2, p2 = fb.fewbit_fwd(t, z)
            torch.cuda.synchronize()
            assert torch.equal(p1, p2) and torch.equal(y1.view(torch.uint8), y2.view(torch.uint8)), (seed, dtype, act, bits, rows, cols, mode)
        fb.fewbit_set_option("fwd_table", "auto")


# --------------------------------------------------------------------------
# bias in front of the activation
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["bf16", "f16", "f32"])
def test_forward_with_bias_matches_the_oracle(dtype, table_mode):
    """f(x + bias): the oracle adds the bias (exact sum, one rounding) and runs its forward half on
    the sum; codes and grad_in bit-exact, y within 2 ulp, for every bucketize variant."""
    rows, cols = 37, 3072
    gen = torch.Generator(device=DEV).manual_seed(11)
    x = (torch.randn(rows, cols, device=DEV, generator=gen) * 1.5).to(TORCH_DT[dtype])
    b = (torch.randn(cols, device=DEV, generator=gen) * 0.7).to(TORCH_DT[dtype])
    b[:4] = torch.tensor([0.0, -0.0, 1e-3, -40.0], device=DEV).to(TORCH_DT[dtype])
    x[0, :8] = torch.tensor([0.0, -0.0, 1.0, -1.0, 65000.0, -1e-7, 3.0, 0.5], device=DEV).to(TORCH_DT[dtype])
    g = torch.randn(rows, cols, device=DEV, generator=gen).to(TORCH_DT[dtype])
    z_np = oracle.bias_add(np_bits(x).reshape(rows, cols), np_bits(b)).reshape(-1)
    for act, bits in (("gelu", 1), ("silu", 2), ("sigmoid", 3), ("gelu", 4), ("tanh", 4)):
        t = table(act, bits)
        s_np, lev_np = t.arrays()
        y, pk = fb.fewbit_fwd_bias(t, x, b)
        gi = fb.fewbit_bwd(t, pk, g)
        torch.cuda.synchronize()
        y_ref, p_ref = oracle.fwd(act, bits, s_np, z_np)
        gi_ref = oracle.bwd(bits, lev_np, p_ref, np_bits(g).reshape(-1))
        assert np.array_equal(np_bits(pk).view(np.uint32), p_ref), (dtype, act, bits)
        assert np.array_equal(np_bits(gi).reshape(-1).view(gi_ref.dtype), gi_ref), (dtype, act, bits)
        ok = finite_mask(z_np)
        assert ulp_distance(np_bits(y).reshape(-1)[ok], y_ref[ok]).max() <= 2, (dtype, act, bits)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("rows,cols", [(3, 8), (129, 40), (77, 1000), (5, 11008), (1, 1048), (1031, 1016)])
def test_forward_with_bias_on_row_lengths_that_are_not_whole_warp_blocks(dtype, rows, cols, table_mode):
    """Row lengths that are multiples of 8 only: warp-blocks straddle row ends, the last one is
    ragged and takes the scalar path; codes and grad_in bit-exact, y within 2 ulp."""
    gen = torch.Generator(device=DEV).manual_seed(rows * 131 + cols)
    x = (torch.randn(rows, cols, device=DEV, generator=gen) * 1.5).to(TORCH_DT[dtype])
    b = torch.randn(cols, device=DEV, generator=gen).to(TORCH_DT[dtype])
    g = torch.randn(rows, cols, device=DEV, generator=gen).to(TORCH_DT[dtype])
    z_np = oracle.bias_add(np_bits(x).reshape(rows, cols), np_bits(b)).reshape(-1)
    for act, bits in (("silu", 1), ("gelu", 3), ("tanh", 4)):
        t = table(act, bits)
        s_np, lev_np = t.arrays()
        y, pk = fb.fewbit_fwd_bias(t, x, b)
        gi = fb.fewbit_bwd(t, pk, g)
        torch.cuda.synchronize()
        y_ref, p_ref = oracle.fwd(act, bits, s_np, z_np)
        gi_ref = oracle.bwd(bits, lev_np, p_ref, np_bits(g).reshape(-1))
        assert np.array_equal(np_bits(pk).view(np.uint32), p_ref), (dtype, rows, cols, act, bits)
        assert np.array_equal(np_bits(gi).reshape(-1).view(gi_ref.dtype), gi_ref)
        assert ulp_distance(np_bits(y).reshape(-1), y_ref).max() <= 2


@pytest.mark.parametrize("dtype", ["bf16", "f16"])
def test_bias_sum_over_every_pattern_against_random_patterns(dtype):
    """Every 16-bit pattern as x (subnormals, infinities, NaNs included), eight rows rolled against
    a bias of random patterns: the kernel's sum is the oracle's (exact sum, one rounding), seen
    through the codes (bit-exact) and y (within 2 ulp where the sum is finite)."""
    cols, rows = 65536, 8
    rng = np.random.default_rng(77)
    pat = np.arange(cols, dtype=np.uint16)
    x_bits = np.stack([np.roll(pat, 8191 * r) for r in range(rows)])
    b_bits = rng.integers(0, 65536, cols).astype(np.uint16)
    b_bits[:16] = [0x0000, 0x8000, 0x0001, 0x8001, 0x007f, 0x0080, 0x7f7f, 0xff7f, 0x3f80, 0xbf80, 0x0400, 0x8400, 0x7bff, 0xfbff, 0x3c00, 0xbc00]
    tdt = TORCH_DT[dtype]
    x = torch.from_numpy(x_bits.view(np.int16)).to(DEV).view(tdt)
    b = torch.from_numpy(b_bits.view(np.int16)).to(DEV).view(tdt)
    as_np = (lambda a: a) if dtype == "bf16" else (lambda a: a.view(np.float16))
    z_np = oracle.bias_add(as_np(x_bits), as_np(b_bits)).reshape(-1)
    t = table("silu", 4)
    s_np, _ = t.arrays()
    y, pk = fb.fewbit_fwd_bias(t, x, b)
    torch.cuda.synchronize()
    y_ref, p_ref = oracle.fwd("silu", 4, s_np, z_np)
    assert np.array_equal(np_bits(pk).view(np.uint32), p_ref)
    ok = finite_mask(z_np)
    assert ulp_distance(np_bits(y).reshape(-1)[ok], y_ref[ok]).max() <= 2
    # the sum itself, bit for bit: leaky ReLU returns a positive argument unchanged; then the mirror image
    tl = table("leaky_relu", 1)
    for flip in (0x0000, 0x8000):
        xf = torch.from_numpy((x_bits ^ np.uint16(flip)).view(np.int16)).to(DEV).view(tdt)
        bf = torch.from_numpy((b_bits ^ np.uint16(flip)).view(np.int16)).to(DEV).view(tdt)
        zf = oracle.bias_add(as_np(x_bits ^ np.uint16(flip)), as_np(b_bits ^ np.uint16(flip))).reshape(-1)
        yl, _ = fb.fewbit_fwd_bias(tl, xf, bf)
        torch.cuda.synchronize()
        zv = bf16_bits_to_f32(zf) if dtype == "bf16" else zf.astype(np.float32)
        pos = np.isfinite(zv) & (zv > 0)
        assert pos.sum() > 100000
        assert np.array_equal(np_bits(yl).reshape(-1).view(np.uint16)[pos], zf.view(np.uint16)[pos])


def test_autograd_layer_with_bias_gives_the_column_sums():
    rows, cols = 48, 2056
    x = torch.randn(rows, cols, device=DEV, dtype=torch.bfloat16, requires_grad=True)
    bias = (torch.randn(cols, device=DEV) * 0.5).bfloat16().requires_grad_(True)
    layer = fb.FewBitActivation("gelu", bits=3)
    y = layer(x, bias)
    g = torch.randn_like(y)
    y.backward(g)
    t = layer.table
    z = (x.detach().float() + bias.detach().float()[None, :]).bfloat16()
    y_ref, pk = fb.fewbit_fwd(t, z)
    gi_ref = fb.fewbit_bwd(t, pk, g)
    assert torch.equal(y.detach().view(torch.int16), y_ref.view(torch.int16))
    assert torch.equal(x.grad.view(torch.int16), gi_ref.view(torch.int16))
    assert torch.equal(bias.grad, gi_ref.float().sum(0).bfloat16())


def test_forward_with_bias_on_a_large_tensor_in_place_and_its_argument_checks():
    rows, cols = 8192, 4096                               # 2^25 elements: the dynamically distributed table variant at 4 bits
    t = table("gelu", 4)
    x = torch.randn(rows, cols, device=DEV).bfloat16()
    b = torch.randn(cols, device=DEV).bfloat16()
    y, pk = fb.fewbit_fwd_bias(t, x, b)
    z = (x.float() + b.float()[None, :]).bfloat16()       # binary32 sum, one rounding: the same value
    y2, pk2 = fb.fewbit_fwd(t, z)
    torch.cuda.synchronize()
    assert torch.equal(pk, pk2) and torch.equal(y.view(torch.int16), y2.view(torch.int16))
    xi = x.clone()
    fb.fewbit_fwd_bias(t, xi, b, y=xi)                    # y aliases x
    torch.cuda.synchronize()
    assert torch.equal(xi.view(torch.int16), y.view(torch.int16))
    compare_sampled("gelu", 4, z.reshape(-1), z.reshape(-1), y.reshape(-1), pk, fb.fewbit_bwd(t, pk, z.reshape(-1)), "bias, large")
    with pytest.raises(fb.FewbitError) as e:              # a row must be a whole number of 8-element lane-chunks
        fb.fewbit_fwd_bias(t, x[:, :1004].contiguous(), b[:1004].contiguous())
    assert e.value.status == 2
    with pytest.raises(ValueError):
        fb.fewbit_fwd_bias(t, x, b[:1024].contiguous())
    with pytest.raises(fb.FewbitError) as e:              # no folded tables with a bias
        fb.fewbit_fwd_bias(fb.fewbit_table_create_folded("tanh", 2), x, b)
    assert e.value.status == 2
    # binary32 at a size where its table variant is distributed dynamically (3 and 4 bits)
    xf = torch.randn(4096, 4096, device=DEV)
    bf = torch.randn(4096, device=DEV)
    zf = xf + bf[None, :]                                 # one IEEE binary32 addition per element
    for act, bits in (("sigmoid", 3), ("silu", 4)):
        tf = table(act, bits)
        y1, p1 = fb.fewbit_fwd_bias(tf, xf, bf)
        y2, p2 = fb.fewbit_fwd(tf, zf)
        torch.cuda.synchronize()
        assert torch.equal(p1, p2) and torch.equal(y1.view(torch.int32), y2.view(torch.int32)), (act, bits)


def test_more_than_2_to_the_32_elements():
    """Element and word indices beyond 32 bits: 2^32 + 3149 bfloat16 elements (about 28 GB on the
    device), 1 bit (search variant) and 4 bits (table variant, dynamically distributed); sampled
    blocks include the ones that straddle element 2^32 and the ragged tail."""
    n = (1 << 32) + 3 * 1024 + 77
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * 2 ** 30:
        pytest.skip("needs ~28 GB of free device memory")
    x = torch.empty(n, device=DEV, dtype=torch.bfloat16)
    gen = torch.Generator(device=DEV).manual_seed(5)
    step = 1 << 28
    for e0 in range(0, n, step):
        m = min(step, n - e0)
        x[e0:e0 + m] = torch.randn(m, device=DEV, generator=gen).mul_(1.5).bfloat16()
    near = [(1 << 32) - 4096, (1 << 32) - 32, 1 << 32, (1 << 31) - 4096, 1 << 31]
    for bits in (1, 4):
        t = table("silu", bits)
        y, pk = fb.fewbit_fwd(t, x)
        gi = fb.fewbit_bwd(t, pk, x)                # the input doubles as the incoming gradient
        torch.cuda.synchronize()
        compare_sampled("silu", bits, x, x, y, pk, gi, f"2^32+ k={bits}", blocks=16, seed=bits, also_at=near)
        del y, pk, gi


# --------------------------------------------------------------------------
# edge cases
# --------------------------------------------------------------------------
@pytest.fixture(params=["auto", "always", "never"])
def table_mode(request):
    """Runs a test under each bucketize variant: size-based choice, shared-memory
    code table forced on (where the table has one), forced off."""
    fb.fewbit_set_option("fwd_table", request.param)
    yield request.param
    fb.fewbit_set_option("fwd_table", "auto")



@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_ragged_sizes(dtype, bits, table_mode):
    gen = torch.Generator(device=DEV).manual_seed(11)
    for n in [1, 7, 31, 32, 33, 255, 256, 257, 1023, 1024, 1025, 2047, 2048 + 33, 5 * 1024 + 1000, 9999]:
        x = (torch.randn(n, generator=gen, device=DEV) * 2).to(TORCH_DT[dtype])
        g = torch.randn(n, generator=gen, device=DEV).to(TORCH_DT[dtype])
        y, p, gi = run_gpu("silu", bits, x, g)
        compare_full("silu", bits, x, g, y, p, gi, f"ragged n={n}")


def test_empty_input_is_a_no_op():
    t = table("gelu", 2)
    x = torch.empty(0, device=DEV)
    before = fb.fewbit_launch_count()
    y, p = fb.fewbit_fwd(t, x)
    gi = fb.fewbit_bwd(t, p, x)
    assert y.numel() == 0 and p.numel() == 0 and gi.numel() == 0
    assert fb.fewbit_launch_count() == before


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_in_place_aliasing(dtype, table_mode):
    gen = torch.Generator(device=DEV).manual_seed(5)
    n = 70001
    x = torch.randn(n, generator=gen, device=DEV).to(TORCH_DT[dtype])
    g = torch.randn(n, generator=gen, device=DEV).to(TORCH_DT[dtype])
    for bits in (1, 3):
        y, p, gi = run_gpu("tanh", bits, x, g, inplace=True)
        compare_full("tanh", bits, x, g, y, p, gi, "in place")


@pytest.mark.parametrize("act", wl.ACTIVATIONS + wl.EXTRA_ACTIVATIONS)
def test_every_bf16_pattern(act, table_mode):
    """All 65 536 bfloat16 inputs: codes for every pattern (NaN and infinities
    included), y for every finite input."""
    h = torch.arange(65536, dtype=torch.int32).to(torch.int16).view(torch.bfloat16).to(DEV)
    g = torch.ones_like(h)
    for bits in (1, 4):
        y, p, gi = run_gpu(act, bits, h, g)
        compare_full(act, bits, h, g, y, p, gi, f"all bf16 {act}")


@pytest.mark.parametrize("act", wl.ACTIVATIONS + wl.EXTRA_ACTIVATIONS)
def test_f32_values_around_every_boundary_and_in_the_tails(act, table_mode):
    pieces = []
    for bits in (1, 2, 3, 4):
        s, _ = table(act, bits).arrays()
        pieces += [s, np.nextafter(s, np.float32(np.inf)), np.nextafter(s, np.float32(-np.inf))]
    rng = np.random.default_rng(7)
    mags = (10.0 ** rng.uniform(-44, 2.2, 20000)).astype(np.float32)
    pieces += [mags, -mags, np.linspace(-20, 20, 40001, dtype=np.float32),
               np.array([0.0, -0.0, 1e-45, -1e-45, 88.0, -88.0, 100.0, -100.0, -103.9, 3e38, -3e38], dtype=np.float32)]
    x_np = np.concatenate(pieces)
    x = torch.from_numpy(x_np).to(DEV)
    g = torch.ones_like(x)
    for bits in (1, 2, 3, 4):
        y, p, gi = run_gpu(act, bits, x, g)
        compare_full(act, bits, x, g, y, p, gi, f"special f32 {act} k={bits}")


def test_gradient_specials_are_bit_exact():
    """Denormal, huge and signed-zero gradients: one binary32 multiply, one rounding."""
    rng = np.random.default_rng(3)
    n = 40000
    gf = (rng.standard_normal(n) * 10.0 ** rng.uniform(-44, 37, n)).astype(np.float32)
    gf[:4] = [0.0, -0.0, 1e-45, -1e-45]
    x = torch.from_numpy((rng.standard_normal(n) * 2).astype(np.float32)).to(DEV)
    for dtype in ("f32", "bf16"):
        g = torch.from_numpy(gf).to(DEV).to(TORCH_DT[dtype])
        xs = x.to(TORCH_DT[dtype])
        for bits in (2, 4):
            y, p, gi = run_gpu("gelu", bits, xs, g)
            compare_full("gelu", bits, xs, g, y, p, gi, f"grad specials {dtype}")


def test_injected_table_with_equal_boundaries(table_mode):
    s = np.array([-1.0, 0.0, 0.0, 0.0, 0.5, 0.5, 3.0], dtype=np.float32)
    lev = np.linspace(-1, 1, 8).astype(np.float32)
    t = fb.fewbit_table_from_arrays("elu", 3, s, lev)
    x = torch.linspace(-4, 4, 8193, device=DEV)
    g = torch.ones_like(x)
    y, p = fb.fewbit_fwd(t, x)
    gi = fb.fewbit_bwd(t, p, g)
    torch.cuda.synchronize()
    y_ref, p_ref = oracle.fwd("elu", 3, s, np_bits(x))
    gi_ref = oracle.bwd(3, lev, p_ref, np_bits(g))
    assert np.array_equal(np_bits(p).view(np.uint32), p_ref)
    assert np.array_equal(np_bits(gi), gi_ref)


@pytest.mark.parametrize("act", ["sigmoid", "tanh"])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_folded_tables(act, dtype, table_mode):
    """Even-derivative fold: codes from |x| against the oracle, every bit width, every variant."""
    gen = torch.Generator(device=DEV).manual_seed(21)
    n = 3 * 2 ** 20 + 77
    x = (torch.randn(n, generator=gen, device=DEV) * 2).to(TORCH_DT[dtype])
    x[:6] = torch.tensor([0.0, -0.0, float("inf"), float("-inf"), float("nan"), -1e-30], device=DEV).to(TORCH_DT[dtype])
    g = torch.randn(n, generator=gen, device=DEV).to(TORCH_DT[dtype])
    for bits in (1, 2, 3, 4):
        t = fb.fewbit_table_create_folded(act, bits)
        s, lev = t.arrays()
        x[6:6 + s.size] = torch.from_numpy(s).to(DEV).to(TORCH_DT[dtype])
        x[40:40 + s.size] = -torch.from_numpy(s).to(DEV).to(TORCH_DT[dtype])
        y, p = fb.fewbit_fwd(t, x)
        gi = fb.fewbit_bwd(t, p, g)
        torch.cuda.synchronize()
        y_ref, p_ref = oracle.fwd(act, bits, s, np_bits(x), fold=True)
        gi_ref = oracle.bwd(bits, lev, p_ref, np_bits(g))
        assert np.array_equal(np_bits(p).view(np.uint32), p_ref), (act, dtype, bits)
        assert np.array_equal(np_bits(gi).view(gi_ref.dtype), gi_ref), (act, dtype, bits)
        ok = finite_mask(np_bits(x))
        assert ulp_distance(np_bits(y)[ok], y_ref[ok]).max() <= 2


def test_folded_table_at_table_variant_size():
    """Large enough for the shared-memory code table to be chosen on its own (bf16, 4 bits)."""
    n = 2 ** 27
    gen = torch.Generator(device=DEV).manual_seed(22)
    x = (torch.randn(n, generator=gen, device=DEV) * 2).bfloat16()
    t = fb.fewbit_table_create_folded("sigmoid", 4)      # 27 waves: the table is this activation's choice from 24 on
    s, _ = t.arrays()
    y, p = fb.fewbit_fwd(t, x)
    torch.cuda.synchronize()
    for e0 in (0, 12345 * 1024, n - 8192):
        _, p_ref = oracle.fwd("sigmoid", 4, s, np_bits(x[e0:e0 + 8192]), fold=True)
        assert np.array_equal(np_bits(p[e0 // 8:e0 // 8 + 1024]).view(np.uint32), p_ref)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_boundaries_closer_than_a_table_cell(dtype, table_mode):
    """Boundaries a few binary32 ulps apart land in one cell of the binary32 code table (the warp
    must fall back to the search there) and round to one bfloat16 (the packed search must still
    count them separately)."""
    base = np.float32(0.7431)
    s = np.array([-1.0, base, np.nextafter(base, np.float32(1)), np.nextafter(np.nextafter(base, np.float32(1)), np.float32(1)),
                  1.5, 1.5, 2.0], dtype=np.float32)
    lev = np.arange(8, dtype=np.float32)
    t = fb.fewbit_table_from_arrays("silu", 3, s, lev)
    near = np.concatenate([np.nextafter(s, np.float32(-9)), s, np.nextafter(s, np.float32(9))])
    x_np = np.concatenate([near, np.linspace(-3, 3, 50001).astype(np.float32), np.array([np.inf, -np.inf, np.nan], np.float32)])
    x = torch.from_numpy(x_np).to(DEV).to(TORCH_DT[dtype])
    g = torch.ones_like(x)
    y, p = fb.fewbit_fwd(t, x)
    gi = fb.fewbit_bwd(t, p, g)
    torch.cuda.synchronize()
    _, p_ref = oracle.fwd("silu", 3, s, np_bits(x))
    gi_ref = oracle.bwd(3, lev, p_ref, np_bits(g))
    assert np.array_equal(np_bits(p).view(np.uint32), p_ref)
    assert np.array_equal(np_bits(gi).view(gi_ref.dtype), gi_ref)


def test_misaligned_device_buffers_are_rejected():
    t = table("gelu", 2)
    x = torch.zeros(4096 + 8, device=DEV)
    with pytest.raises(fb.FewbitError) as e:
        fb.fewbit_fwd(t, x[1:4097])                       # 4 bytes off: below the 16-byte rule
    assert e.value.status == 3
    with pytest.raises(fb.FewbitError) as e:
        fb.fewbit_fwd(t, x[2:4098])
    assert e.value.status == 3
    h = torch.zeros(4096 + 8, device=DEV, dtype=torch.bfloat16)
    with pytest.raises(fb.FewbitError) as e:
        fb.fewbit_fwd(t, h[4:4100])                       # 8 bytes off
    assert e.value.status == 3


@pytest.mark.parametrize("dtype", ["bf16", "f16", "f32"])
@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_buffers_at_the_minimum_alignment(dtype, bits, table_mode):
    """The rule of the boundary: element buffers 16-byte aligned, packed words 4-byte aligned.  Every
    buffer is a view that starts 16 bytes (elements) or 4, 8, 12 bytes (packed) into a 256-byte aligned
    allocation, with canaries on both sides; codes and grad_in bit-exact with the oracle, y within 2 ulp.
    Sizes cover the ragged path alone, whole warp-blocks and the table variants' sizes."""
    tdt = TORCH_DT[dtype]
    es = torch.empty(0, dtype=tdt).element_size()
    off = 16 // es
    gen = torch.Generator(device=DEV).manual_seed(17 + bits)
    t = table("sigmoid", bits)
    for n, poff in ((1000, 1), (5 * 1024 + 77, 2), ((1 << 22) + 1024 * 3 + 5, 3), ((1 << 23) + 9, 1)):
        words = fb.fewbit_packed_bytes(n, bits) // 4
        x = (torch.randn(n + off, generator=gen, device=DEV) * 2).to(tdt)[off:]
        g = torch.randn(n + off, generator=gen, device=DEV).to(tdt)[off:]
        ybuf = torch.full((n + 2 * 128 + off,), 777.0, dtype=tdt, device=DEV)
        gbuf = torch.full((n + 2 * 128 + off,), 777.0, dtype=tdt, device=DEV)
        pbuf = torch.full((words + 2 * 64 + poff,), 0x5A5A5A5A, dtype=torch.int32, device=DEV)
        y, gi, pk = ybuf[128 + off:128 + off + n], gbuf[128 + off:128 + off + n], pbuf[64 + poff:64 + poff + words]
        assert x.data_ptr() % 32 == 16 and y.data_ptr() % 32 == 16 and pk.data_ptr() % 16 == 4 * poff
        fb.fewbit_fwd(t, x, y, pk)
        fb.fewbit_bwd(t, pk, g, gi)
        torch.cuda.synchronize()
        for buf, lo, m, fill in ((ybuf, 128 + off, n, 777.0), (gbuf, 128 + off, n, 777.0), (pbuf, 64 + poff, words, 0x5A5A5A5A)):
            assert bool((buf[:lo] == fill).all()) and bool((buf[lo + m:] == fill).all()), "wrote outside the buffer"
        compare_full("sigmoid", bits, x, g, y, pk, gi, f"min alignment {dtype} k={bits} n={n}")
        # the same call with the bias in front, the bias view 16 bytes in as well
        cols = 8 * 25
        rows = n // cols
        if rows:
            m = rows * cols
            b = torch.randn(cols + off, generator=gen, device=DEV).to(tdt)[off:]
            z = (x[:m].float().view(rows, cols) + b.float()[None, :]).to(tdt).reshape(-1)
            fb.fewbit_fwd_bias(t, x[:m].view(rows, cols), b, y[:m].view(rows, cols), pk)
            y2, p2 = fb.fewbit_fwd(t, z.contiguous())
            torch.cuda.synchronize()
            mw = fb.fewbit_packed_bytes(m, bits) // 4
            assert torch.equal(pk[:mw], p2) and torch.equal(y[:m].view(torch.uint8), y2.view(torch.uint8))


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_shards_cut_on_32_elements(dtype):
    """A flat tensor cut on multiples of 32 elements: each shard's x, y and packed views satisfy the
    alignment rule as they are, and the shards written side by side into ONE y and ONE packed buffer
    are the single-launch result."""
    tdt = TORCH_DT[dtype]
    n = (1 << 21) + 32 * 37 + 11
    x = (torch.randn(n, device=DEV) * 1.5).to(tdt)
    g = torch.randn(n, device=DEV).to(tdt)
    for bits in (1, 2, 3, 4):
        t = table("gelu", bits)
        y, pk = fb.fewbit_fwd(t, x)
        gi = fb.fewbit_bwd(t, pk, g)
        for world in (3, 7):
            y2, p2, gi2 = torch.zeros_like(y), torch.zeros_like(pk), torch.zeros_like(gi)
            for rank in range(world):
                lo, hi = wl.shard_range(n, rank, world, align=32)
                assert lo % 32 == 0
                w0, w1 = lo // 32 * bits, fb.fewbit_packed_bytes(hi, bits) // 4
                fb.fewbit_fwd(t, x[lo:hi], y2[lo:hi], p2[w0:w1])
                fb.fewbit_bwd(t, p2[w0:w1], g[lo:hi], gi2[lo:hi])
            torch.cuda.synchronize()
            assert torch.equal(p2, pk), (dtype, bits, world)
            assert torch.equal(y2.view(torch.uint8), y.view(torch.uint8))
            assert torch.equal(gi2.view(torch.uint8), gi.view(torch.uint8))


# --------------------------------------------------------------------------
# the ragged tail has exactly one owner, also in place
# --------------------------------------------------------------------------
def _tail_sizes():
    # n = k * 1024 + 5: the partial warp-block sits at every offset 0 .. 11 of a 12-warp CTA (and of
    # 4-warp ones); 2^24 + 7 is the sweep's ragged size
    return [k * 1024 + 5 for k in range(60, 72)] + [2 ** 24 + 7]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("bits", [3, 4])
def test_ragged_tail_has_one_owner_and_works_in_place(dtype, bits):
    """y == x with a ragged last warp-block, binary32 and bfloat16, code table forced and size-based,
    static and dynamic partition, CTA widths of 4, 12 and 16 warps: exactly one warp runs the tail
    (counted on the device), and codes, y and grad_in are the oracle's."""
    tdt = TORCH_DT[dtype]
    gen = torch.Generator(device=DEV).manual_seed(3 + bits)
    fb.fewbit_set_option("count_tails", 1)
    fb.fewbit_tail_warp_count(reset=True)
    for act in ("leaky_relu", "sigmoid"):
        t = table(act, bits)
        for n in _tail_sizes():
            x = (torch.randn(n, generator=gen, device=DEV) * 2).to(tdt)
            g = torch.randn(n, generator=gen, device=DEV).to(tdt)
            ref = None
            for mode, queue, iters in (("auto", "auto", 0), ("always", "never", 0), ("always", "auto", 0), ("always", "never", 1),
                                       ("always", "never", 3), ("never", "auto", 0), ("never", "auto", 2)):
                fb.fewbit_set_option("fwd_table", mode)
                fb.fewbit_set_option("fwd_queue", queue)
                fb.fewbit_set_option("fwd_iters", iters)
                y = x.clone()
                pk = torch.full((fb.fewbit_packed_bytes(n, bits) // 4,), 0x5A5A5A5A, dtype=torch.int32, device=DEV)
                fb.fewbit_fwd(t, y, y, pk)                      # in place
                assert fb.fewbit_tail_warp_count(reset=True) == 1, (dtype, bits, act, n, mode, queue, iters)
                if ref is None:
                    gi = g.clone()
                    fb.fewbit_bwd(t, pk, gi, gi)
                    torch.cuda.synchronize()
                    if n < 2 ** 20:
                        compare_full(act, bits, x, g, y, pk, gi, f"in place, ragged, n={n}")
                    else:
                        compare_sampled(act, bits, x, g, y, pk, gi, f"in place, ragged, n={n}", blocks=8, block_elems=4096)
                    ref = (y, pk)
                else:
                    assert torch.equal(pk, ref[1]) and torch.equal(y.view(torch.uint8), ref[0].view(torch.uint8)), \
                        (dtype, bits, act, n, mode, queue, iters)
            # the same sizes through the bias entry point (rows of 8 elements need n % 8 == 0: cut the view)
            m = n // 8 * 8
            b = torch.zeros(8, device=DEV, dtype=tdt)
            fb.fewbit_set_option("fwd_table", "always")
            fb.fewbit_set_option("fwd_queue", "never")
            fb.fewbit_set_option("fwd_iters", 0)
            yb = x[:m].clone().view(-1, 8)
            pb = torch.empty(fb.fewbit_packed_bytes(m, bits) // 4, dtype=torch.int32, device=DEV)
            fb.fewbit_fwd_bias(t, yb, b, yb, pb)
            assert fb.fewbit_tail_warp_count(reset=True) == (1 if m % 1024 else 0)
            y0, p0 = fb.fewbit_fwd(t, x[:m].contiguous())
            assert fb.fewbit_tail_warp_count(reset=True) == (1 if m % 1024 else 0)
            torch.cuda.synchronize()
            assert torch.equal(pb, p0) and torch.equal(yb.view(torch.uint8).reshape(-1), y0.view(torch.uint8).reshape(-1))


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_tile_mode_gives_the_same_stream(dtype, bits):
    """Small tensors are processed a 256-element tile per warp (the quad of lanes assembles the words
    by shuffle) instead of a 1024-element warp-block.  Forced on at every size class -- ragged below
    one tile, whole tiles, tails at every 32-element offset of a tile, a few hundred tiles -- it gives
    the oracle's codes and grad_in and y within 2 ulp, the bytes of the warp-block path, in place as
    well, with the bias in front as well, and exactly one warp runs the ragged tail."""
    tdt = TORCH_DT[dtype]
    gen = torch.Generator(device=DEV).manual_seed(29 + bits)
    fb.fewbit_set_option("count_tails", 1)
    fb.fewbit_tail_warp_count(reset=True)
    sizes = [1, 31, 32, 33, 255, 256, 257, 511, 1023, 1024, 1025, 2048 + 33, 9999, 70001, (1 << 18) + 256 * 3]
    sizes += [256 * 5 + 32 * k + 3 for k in range(8)]
    for act in ("gelu", "tanh"):
        t = table(act, bits)
        for n in sizes:
            x = (torch.randn(n, generator=gen, device=DEV) * 2).to(tdt)
            g = torch.randn(n, generator=gen, device=DEV).to(tdt)
            fb.fewbit_set_option("fwd_tile", "never")
            y0, p0 = fb.fewbit_fwd(t, x)
            fb.fewbit_tail_warp_count(reset=True)
            fb.fewbit_set_option("fwd_tile", "always")
            words = fb.fewbit_packed_bytes(n, bits) // 4
            pbuf, pk, ppad = guarded(words, torch.int32, 0x5A5A5A5A)
            ybuf, y, ypad = guarded(n, tdt, 777.0)
            fb.fewbit_fwd(t, x, y, pk)
            assert fb.fewbit_tail_warp_count(reset=True) == (1 if n % 256 else 0), (dtype, bits, act, n)
            check_guards(ybuf, n, ypad, 777.0)
            check_guards(pbuf, words, ppad, 0x5A5A5A5A)
            assert torch.equal(pk, p0) and torch.equal(y.view(torch.uint8), y0.view(torch.uint8)), (dtype, bits, act, n)
            xi = x.clone()
            pi = torch.empty_like(p0)
            fb.fewbit_fwd(t, xi, xi, pi)                                  # in place
            assert torch.equal(pi, p0) and torch.equal(xi.view(torch.uint8), y0.view(torch.uint8)), (dtype, bits, act, n)
            if n <= 70001:
                gi = fb.fewbit_bwd(t, pk, g)
                compare_full(act, bits, x, g, y, pk, gi, f"tile mode {dtype} k={bits} {act} n={n}")
            for cols in (8, 200, 1024):                                   # rows shorter than, straddling and longer than a tile
                rows = n // cols
                if rows:
                    m = rows * cols
                    bias = torch.randn(cols, generator=gen, device=DEV).to(tdt)
                    fb.fewbit_set_option("fwd_tile", "never")
                    yb0, pb0 = fb.fewbit_fwd_bias(t, x[:m].view(rows, cols), bias)
                    fb.fewbit_set_option("fwd_tile", "always")
                    yb1, pb1 = fb.fewbit_fwd_bias(t, x[:m].view(rows, cols), bias)
                    assert torch.equal(pb0, pb1) and torch.equal(yb0.view(torch.uint8), yb1.view(torch.uint8)), (dtype, bits, act, n, cols)
    fb.fewbit_tail_warp_count(reset=True)


@pytest.mark.parametrize("warps,iters", [(1, 0), (2, 5), (0, 1), (0, 64), (16, 2), (3, 0)])
def test_launch_geometry_overrides_do_not_change_the_result(warps, iters):
    """FEWBIT_OPT_FWD_WARPS / FEWBIT_OPT_FWD_ITERS only reshape the grid (a single-warp CTA included):
    same y and packed words as the default launch, bfloat16 at 4 bits (shared threshold-pair table)
    and binary32."""
    for dtype, act, bits in (("bf16", "silu", 4), ("bf16", "gelu", 3), ("f32", "tanh", 4), ("f16", "elu", 4)):
        t = table(act, bits)
        for n in (70001, (1 << 21) + 1029):
            x = (torch.randn(n, device=DEV) * 2).to(TORCH_DT[dtype])
            fb.fewbit_set_option("fwd_table", "never")
            y0, p0 = fb.fewbit_fwd(t, x)
            fb.fewbit_set_option("fwd_warps", warps)
            fb.fewbit_set_option("fwd_iters", iters)
            y1, p1 = fb.fewbit_fwd(t, x)
            fb.fewbit_set_option("fwd_warps", 0)
            fb.fewbit_set_option("fwd_iters", 0)
            torch.cuda.synchronize()
            assert torch.equal(p0, p1) and torch.equal(y0.view(torch.uint8), y1.view(torch.uint8)), (dtype, act, bits, n)


def test_runs_on_a_side_stream():
    t = table("silu", 4)
    x = torch.randn(1 << 20, device=DEV).bfloat16()
    g = torch.randn(1 << 20, device=DEV).bfloat16()
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(st):
        y, p = fb.fewbit_fwd(t, x)
        gi = fb.fewbit_bwd(t, p, g)
    st.synchronize()
    compare_full("silu", 4, x, g, y, p, gi, "side stream")


@pytest.mark.parametrize("bits", [3, 4])
def test_dynamic_table_variant_on_concurrent_streams(bits):
    """The table variant of the 16-bit types hands out warp-blocks through leased work counters.
    Three streams at once, twice each (a stream reuses its own counters, different streams must
    not share any): every launch gives exactly what the search variant gives on the same input,
    and that agrees with the oracle on sampled blocks."""
    n = (1 << 25) + 4097
    t = table("gelu", bits)
    gen = torch.Generator(device=DEV).manual_seed(31 + bits)
    xs = [torch.randn(n, device=DEV, generator=gen).bfloat16() for _ in range(3)]
    fb.fewbit_set_option("fwd_table", "never")
    refs = [fb.fewbit_fwd(t, x) for x in xs]
    torch.cuda.synchronize()
    g = torch.ones(n, device=DEV).bfloat16()
    compare_sampled("gelu", bits, xs[0], g, refs[0][0], refs[0][1], fb.fewbit_bwd(t, refs[0][1], g), "search variant")
    fb.fewbit_set_option("fwd_table", "always")
    streams = [torch.cuda.Stream() for _ in xs]
    outs = []
    for rep in range(2):
        for x, st in zip(xs, streams):
            st.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(st):
                outs.append(fb.fewbit_fwd(t, x))
    for st in streams:
        st.synchronize()
    for i, (y, pk) in enumerate(outs):
        y_ref, p_ref = refs[i % 3]
        assert torch.equal(pk, p_ref), f"codes differ, launch {i}"
        assert torch.equal(y.view(torch.int16), y_ref.view(torch.int16)), f"y differs, launch {i}"


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_dynamic_and_static_partition_agree_on_whole_arrays(dtype):
    """Every element and every packed word of the dynamically distributed table variant equals the
    statically partitioned one (a warp-block dropped or done twice would show), ragged tail included."""
    n = (1 << 24) + 4097
    x = (torch.randn(n, device=DEV) * 2).to(TORCH_DT[dtype])
    fb.fewbit_set_option("fwd_table", "always")
    for act in ("sigmoid", "gelu"):
        for bits in (3, 4):
            t = table(act, bits)
            fb.fewbit_set_option("fwd_queue", "never")
            y0, p0 = fb.fewbit_fwd(t, x)
            fb.fewbit_set_option("fwd_queue", "auto")
            y1, p1 = fb.fewbit_fwd(t, x)
            torch.cuda.synchronize()
            assert torch.equal(p0, p1), (dtype, act, bits)
            assert torch.equal(y0.view(torch.uint8), y1.view(torch.uint8)), (dtype, act, bits)


def test_more_streams_than_work_counter_sets_from_several_host_threads():
    """24 streams driven by 6 host threads, two table-variant launches each, nothing waited for in
    between: more launches in flight than there are sets of work counters, so some take the static
    partition.  Every result equals the search variant's."""
    n = (1 << 23) + 1024 * 5 + 3
    t = table("gelu", 4)
    x = torch.randn(n, device=DEV).mul_(1.7).bfloat16()
    fb.fewbit_set_option("fwd_table", "never")
    y_ref, p_ref = fb.fewbit_fwd(t, x)
    torch.cuda.synchronize()
    fb.fewbit_set_option("fwd_table", "always")
    streams = [torch.cuda.Stream() for _ in range(24)]
    outs = [None] * 48

    def drive(k):
        torch.cuda.set_device(DEV)
        for i in range(k, 24, 6):
            with torch.cuda.stream(streams[i]):
                outs[2 * i] = fb.fewbit_fwd(t, x)
                outs[2 * i + 1] = fb.fewbit_fwd(t, x)

    with ThreadPoolExecutor(max_workers=6) as pool:
        list(pool.map(drive, range(6)))
    torch.cuda.synchronize()
    for i, (y, pk) in enumerate(outs):
        assert torch.equal(pk, p_ref), f"codes differ, launch {i}"
        assert torch.equal(y.view(torch.int16), y_ref.view(torch.int16)), f"y differs, launch {i}"


def test_stream_capture_uses_the_static_partition_and_replays():
    """No work counters are leased while a stream is being captured; the captured launch gives the
    same result as the eager (dynamically distributed) one."""
    n = 1 << 25
    t = table("gelu", 4)                            # 6 waves: the table variant is the size-based choice
    x = torch.randn(n, device=DEV).bfloat16()
    y, pk = fb.fewbit_fwd(t, x)                     # eager: also resolves every per-device one-time setting
    torch.cuda.synchronize()
    y2, p2 = torch.zeros_like(y), torch.zeros_like(pk)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        fb.fewbit_fwd(t, x, y2, p2)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(p2, pk)
    assert torch.equal(y2.view(torch.int16), y.view(torch.int16))


def test_dynamic_launch_from_another_thread_while_a_capture_is_in_progress():
    """One host thread captures a CUDA graph in the global capture mode (torch's default) while
    another launches the dynamically distributed table variant on a stream of its own.  Leasing the
    work counters queries CUDA events, which the global mode would refuse from any thread: the
    library makes those calls in the relaxed mode, so the capture stays valid and both results are
    right.  Every buffer is allocated before the capture begins (an allocation would invalidate it)."""
    import threading
    n = (1 << 23) + 4097
    t = table("gelu", 4)
    x = torch.randn(n, device=DEV).mul_(1.3).bfloat16()
    fb.fewbit_set_option("fwd_table", "never")
    y_ref, p_ref = fb.fewbit_fwd(t, x)
    fb.fewbit_set_option("fwd_table", "always")
    # use up every never-used set of work counters, so that the launch below has to query events
    warm = [torch.cuda.Stream() for _ in range(20)]
    for st in warm:
        with torch.cuda.stream(st):
            fb.fewbit_fwd(t, x)
    torch.cuda.synchronize()
    y_cap, p_cap = torch.zeros_like(y_ref), torch.zeros_like(p_ref)
    y_dyn, p_dyn = torch.zeros_like(y_ref), torch.zeros_like(p_ref)
    side = torch.cuda.Stream()
    capturing, launched, errors = threading.Event(), threading.Event(), []

    def other_thread():
        try:
            torch.cuda.set_device(DEV)
            capturing.wait(timeout=60)
            with torch.cuda.stream(side):
                fb.fewbit_fwd(t, x, y_dyn, p_dyn)
        except Exception as exc:                      # pragma: no cover
            errors.append(exc)
        finally:
            launched.set()

    th = threading.Thread(target=other_thread)
    th.start()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        fb.fewbit_fwd(t, x, y_cap, p_cap)
        capturing.set()
        launched.wait(timeout=60)
    th.join()
    assert not errors, errors
    graph.replay()
    torch.cuda.synchronize()
    for y, pk, what in ((y_cap, p_cap, "captured"), (y_dyn, p_dyn, "other thread")):
        assert torch.equal(pk, p_ref), what
        assert torch.equal(y.view(torch.int16), y_ref.view(torch.int16)), what


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_graph_of_forward_and_backward_replays_with_new_inputs(dtype):
    """A captured forward -> backward chain (the backward reads the words the forward wrote, the two
    launches joined by a programmatic dependency) replayed on fresh contents of the same buffers gives
    what the eager calls give."""
    n = (1 << 23) + 1029
    gen = torch.Generator(device=DEV).manual_seed(123)
    x = torch.randn(n, generator=gen, device=DEV).to(TORCH_DT[dtype])
    g = torch.randn(n, generator=gen, device=DEV).to(TORCH_DT[dtype])
    for bits in (1, 3, 4):
        t = table("gelu", bits)
        y, pk = fb.fewbit_fwd(t, x)                 # eager once: per-device one-time settings
        gi = fb.fewbit_bwd(t, pk, g)
        torch.cuda.synchronize()
        y2, p2, gi2 = torch.zeros_like(y), torch.zeros_like(pk), torch.zeros_like(gi)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            fb.fewbit_fwd(t, x, y2, p2)
            fb.fewbit_bwd(t, p2, g, gi2)
        for rep in range(3):
            if rep:
                x.copy_((torch.randn(n, generator=gen, device=DEV) * (1 + rep)).to(x.dtype))
                g.copy_(torch.randn(n, generator=gen, device=DEV).to(g.dtype))
                y, pk = fb.fewbit_fwd(t, x)
                gi = fb.fewbit_bwd(t, pk, g)
            graph.replay()
            torch.cuda.synchronize()
            assert torch.equal(p2, pk), (bits, rep)
            assert torch.equal(y2.view(torch.uint8), y.view(torch.uint8)), (bits, rep)
            assert torch.equal(gi2.view(torch.uint8), gi.view(torch.uint8)), (bits, rep)


# --------------------------------------------------------------------------
# host-buffer entry points
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("pinned", [True, False])
def test_host_entry_points_match_the_oracle(dtype, pinned):
    n = 300000 + 77
    gen = torch.Generator().manual_seed(9)
    x = torch.randn(n, generator=gen).to(TORCH_DT[dtype])
    g = torch.randn(n, generator=gen).to(TORCH_DT[dtype])
    if pinned:
        x, g = x.pin_memory(), g.pin_memory()
    for bits in (1, 3, 4):
        t = table("softplus", bits)
        words = fb.fewbit_packed_bytes(n, bits) // 4
        mk = (lambda *a, **k: torch.empty(*a, **k).pin_memory()) if pinned else torch.empty
        y, gi, p = mk(n, dtype=x.dtype), mk(n, dtype=x.dtype), mk(words, dtype=torch.int32)
        # a workspace for 32768-element chunks forces ten pipeline steps
        ws = torch.empty(fb.fewbit_host_workspace_bytes(32768, x.dtype, bits), dtype=torch.uint8, device=DEV)
        fb.fewbit_fwd_host(t, x, y, p, ws)
        fb.fewbit_bwd_host(t, p, g, gi, ws)
        compare_full("softplus", bits, x, g, y, p, gi, f"host {dtype} k={bits}")


def test_host_entry_points_with_a_small_workspace_equal_the_device_path():
    """A workspace much smaller than the tensor: every pipeline stage is reused several times, with
    every bit width, and the bytes that come back must be those of the single device-resident launch."""
    n = (1 << 23) + 4133
    gen = torch.Generator().manual_seed(99)
    x = torch.randn(n, generator=gen).to(torch.bfloat16).pin_memory()
    g = torch.randn(n, generator=gen).to(torch.bfloat16).pin_memory()
    for bits in (1, 2, 3, 4):
        t = table("gelu", bits)
        words = fb.fewbit_packed_bytes(n, bits) // 4
        y = torch.empty(n, dtype=x.dtype).pin_memory()
        gi = torch.empty(n, dtype=x.dtype).pin_memory()
        p = torch.empty(words, dtype=torch.int32).pin_memory()
        ws = torch.empty(fb.fewbit_host_workspace_bytes(1 << 20, x.dtype, bits), dtype=torch.uint8, device=DEV)
        for _ in range(2):                     # the second pass finds the workspace dirty
            y.fill_(3.0), gi.fill_(3.0), p.fill_(0x55555555)
            fb.fewbit_fwd_host(t, x, y, p, ws)
            fb.fewbit_bwd_host(t, p, g, gi, ws)
            y_d, p_d, gi_d = run_gpu("gelu", bits, x.to(DEV), g.to(DEV))
            assert torch.equal(p, p_d.cpu()), bits
            assert torch.equal(y.view(torch.int16), y_d.cpu().view(torch.int16)), bits
            assert torch.equal(gi.view(torch.int16), gi_d.cpu().view(torch.int16)), bits


# --------------------------------------------------------------------------
# ReLU / SELU and the autograd layer
# --------------------------------------------------------------------------
@pytest.mark.parametrize("act", wl.EXTRA_ACTIVATIONS)
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_relu_and_selu_against_the_oracle(act, dtype):
    gen = torch.Generator(device=DEV).manual_seed(31)
    n = 2 ** 21 + 5
    x = (torch.randn(n, generator=gen, device=DEV) * 2).to(TORCH_DT[dtype])
    g = torch.randn(n, generator=gen, device=DEV).to(TORCH_DT[dtype])
    for bits in (1, 2, 3, 4):
        y, p, gi = run_gpu(act, bits, x, g)
        compare_full(act, bits, x, g, y, p, gi, f"{act} k={bits} {dtype}")


def test_one_bit_relu_layer_is_exactly_relu():
    """Sec. 2, ReLU paragraph: one bit reproduces the derivative, so the layer's gradient equals torch's."""
    layer = fb.FewBitActivation("relu", bits=1)
    x = torch.randn(1 << 18, device=DEV, requires_grad=True)
    x2 = x.detach().clone().requires_grad_(True)
    g = torch.randn_like(x)
    layer(x).backward(g)
    torch.relu(x2).backward(g)
    assert torch.equal(x.grad, x2.grad)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_autograd_layer_matches_the_oracle_and_saves_only_the_codes(dtype):
    bits = 3
    layer = fb.FewBitActivation("gelu", bits=bits)
    x = (torch.randn(64, 1031, device=DEV) * 1.5).to(TORCH_DT[dtype]).requires_grad_(True)
    saved = []
    with torch.autograd.graph.saved_tensors_hooks(lambda t: (saved.append(t), t)[1], lambda t: t):
        y = layer(x)
    assert len(saved) == 1 and saved[0].numel() * 4 == fb.fewbit_packed_bytes(x.numel(), bits)
    g = torch.randn_like(y)
    y.backward(g)
    s, lev = layer.table.arrays()
    y_ref, p_ref = oracle.fwd("gelu", bits, s, np_bits(x.detach().reshape(-1)))
    gi_ref = oracle.bwd(bits, lev, p_ref, np_bits(g.reshape(-1)))
    assert np.array_equal(np_bits(x.grad.reshape(-1)).view(gi_ref.dtype), gi_ref)
    assert ulp_distance(np_bits(y.detach().reshape(-1)), y_ref).max() <= 2


def test_autograd_layer_trains_a_small_mlp():
    """Same initialisation, same data: the 4-bit layer trains like the exact activation."""
    xs = torch.randn(512, 32, device=DEV, generator=torch.Generator(device=DEV).manual_seed(1))
    ys = torch.tanh(xs[:, :4].sum(1, keepdim=True)).detach()
    final = {}
    for name, act in (("fewbit", lambda: fb.FewBitActivation("silu", 4)), ("exact", torch.nn.SiLU)):
        torch.manual_seed(0)
        net = torch.nn.Sequential(torch.nn.Linear(32, 256), act(), torch.nn.Linear(256, 1)).to(DEV)
        opt = torch.optim.SGD(net.parameters(), lr=0.05)
        first = None
        for _ in range(100):
            loss = ((net(xs) - ys) ** 2).mean()
            first = first if first is not None else loss.item()
            opt.zero_grad(); loss.backward(); opt.step()
        final[name] = loss.item()
        assert loss.item() < 0.5 * first
    assert final["fewbit"] < 1.15 * final["exact"]


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_finetuned_normal_weight_table(dtype, table_mode):
    """Off-grid boundaries (Eq. 5 fine-tuning, normal weight): the hot path only sees another table."""
    gen = torch.Generator(device=DEV).manual_seed(41)
    n = 2 ** 20 + 333
    x = torch.randn(n, generator=gen, device=DEV).to(TORCH_DT[dtype])
    g = torch.randn(n, generator=gen, device=DEV).to(TORCH_DT[dtype])
    for bits in (2, 4):
        t = fb.fewbit_table_create_opt("gelu", bits, weight="normal", finetune_iters=500)
        s, lev = t.arrays()
        x[:s.size] = torch.from_numpy(s).to(DEV).to(TORCH_DT[dtype])
        y, p = fb.fewbit_fwd(t, x)
        gi = fb.fewbit_bwd(t, p, g)
        torch.cuda.synchronize()
        _, p_ref = oracle.fwd("gelu", bits, s, np_bits(x))
        gi_ref = oracle.bwd(bits, lev, p_ref, np_bits(g))
        assert np.array_equal(np_bits(p).view(np.uint32), p_ref)
        assert np.array_equal(np_bits(gi).view(gi_ref.dtype), gi_ref)


# --------------------------------------------------------------------------
# IEEE binary16 storage
# --------------------------------------------------------------------------
@pytest.mark.parametrize("act", wl.ACTIVATIONS + wl.EXTRA_ACTIVATIONS)
def test_every_f16_pattern(act, table_mode):
    """All 65 536 binary16 inputs: codes for every pattern, y (2 ulp of binary16) for every finite one."""
    h = torch.arange(65536, dtype=torch.int32).to(torch.int16).view(torch.float16).to(DEV)
    g = torch.ones_like(h)
    for bits in (1, 3, 4):
        y, p, gi = run_gpu(act, bits, h, g)
        compare_full(act, bits, h, g, y, p, gi, f"all f16 {act}")


@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_f16_random_ragged_and_gradient_specials(bits, table_mode):
    gen = torch.Generator(device=DEV).manual_seed(51)
    rng = np.random.default_rng(52)
    for n in (1, 33, 1025, 70001, 2 ** 21 + 9):
        x = (torch.randn(n, generator=gen, device=DEV) * 2).half()
        gf = (rng.standard_normal(n) * 10.0 ** rng.uniform(-8, 4, n)).astype(np.float16)
        g = torch.from_numpy(gf).to(DEV)
        y, p, gi = run_gpu("gelu", bits, x, g)
        compare_full("gelu", bits, x, g, y, p, gi, f"f16 n={n}")
    x = (torch.randn(300001, generator=gen, device=DEV) * 2).half()
    g = torch.randn(300001, generator=gen, device=DEV).half()
    t = fb.fewbit_table_create_folded("tanh", bits)
    s, lev = t.arrays()
    y, p = fb.fewbit_fwd(t, x)
    gi = fb.fewbit_bwd(t, p, g)
    torch.cuda.synchronize()
    y_ref, p_ref = oracle.fwd("tanh", bits, s, np_bits(x), fold=True)
    assert np.array_equal(np_bits(p).view(np.uint32), p_ref)
    assert np.array_equal(np_bits(gi).view(np.uint16), oracle.bwd(bits, lev, p_ref, np_bits(g)).view(np.uint16))
    assert ulp_distance(np_bits(y), y_ref).max() <= 2


def test_f16_at_table_variant_size_and_through_autograd():
    n = 2 ** 27
    gen = torch.Generator(device=DEV).manual_seed(53)
    x = (torch.randn(n, generator=gen, device=DEV) * 2).half()
    g = torch.ones_like(x)
    y, p, gi = run_gpu("silu", 4, x, g)
    compare_sampled("silu", 4, x, g, y, p, gi, "f16 2^27", blocks=8, block_elems=4096, seed=1)
    del y, p, gi, g
    layer = fb.FewBitActivation("gelu", 2)
    xs = x[:100000].clone().requires_grad_(True)
    layer(xs).sum().backward()
    assert xs.grad.dtype == torch.float16 and bool(torch.isfinite(xs.grad).all())


@pytest.mark.parametrize("act", wl.ACTIVATIONS + wl.EXTRA_ACTIVATIONS)
def test_f32_arithmetic_over_all_inputs_against_binary64_on_the_device(act):
    """Every finite binary32 input: the library's binary32 evaluation of the activation is within
    2 ulp of the binary64 evaluation rounded once.  (Device against device: it extends the parity
    tests above, which tie the same arithmetic to the oracle on samples, to the whole input range.)"""
    r = fb.fewbit_f32_activation_scan(act)
    finite = 2 * (0x7F800000)                      # patterns below the infinities, both signs
    assert sum(r["hist"]) == finite
    assert r["hist"][3] == 0 and r["max_ulp"] <= 2, (act, r, hex(r["worst_pattern"]))


def test_f32_scan_agrees_with_the_oracle_on_a_range():
    """The scan's reference (binary64 on the device) and the oracle agree on what the scan reports:
    for a stretch of patterns, the histogram of |y - oracle| recomputed on the host from fewbit_fwd
    matches the one the scan returns."""
    first, count = 0xBF000000, 1 << 16              # 65 536 consecutive inputs from -0.5 downward
    bits_ = np.arange(first, first + count, dtype=np.uint32)
    x = torch.from_numpy(bits_.view(np.float32).copy()).to(DEV)
    for act in ("gelu", "silu", "softplus"):
        t = table(act, 2)
        y, _ = fb.fewbit_fwd(t, x)
        torch.cuda.synchronize()
        s, _ = t.arrays()
        y_ref, _ = oracle.fwd(act, 2, s, np_bits(x))
        d = ulp_distance(np_bits(y), y_ref)
        hist = [int((d == k).sum()) for k in range(3)] + [int((d > 2).sum())]
        r = fb.fewbit_f32_activation_scan(act, first, count)
        assert r["hist"] == hist, (act, r, hist)


@pytest.mark.parametrize("act", wl.ACTIVATIONS + wl.EXTRA_ACTIVATIONS)
def test_f32_scan_reference_is_tied_to_the_oracle_on_every_exponent(act):
    """The scan over all 2^32 inputs compares the library's binary32 arithmetic with a binary64
    evaluation ON THE DEVICE.  This ties that reference to the oracle across the whole range: for every
    binary32 exponent (subnormals included) and both signs, a stretch of 2^13 consecutive mantissas at
    a random offset plus 2^11 scattered ones go through fewbit_fwd; y is within 2 ulp of the oracle on
    all of them, and on the stretches the histogram of |y - oracle| in ulps, recomputed on the host,
    is exactly what the scan reports for the same patterns."""
    rng = np.random.default_rng(1234 + fb.ACTS[act])
    stretch, scattered = 1 << 13, 1 << 11
    firsts, pats = [], []
    for sign in (0, 1):
        for e in range(255):                                 # exponent 255 = infinities and NaNs: not graded
            base = (sign << 31) | (e << 23)
            m0 = int(rng.integers(0, (1 << 23) - stretch + 1))
            firsts.append(base + m0)
            pats.append(base + m0 + np.arange(stretch, dtype=np.int64))
            pats.append(base + rng.integers(0, 1 << 23, scattered))
    bits_all = np.concatenate(pats).astype(np.uint32)
    x = torch.from_numpy(bits_all.view(np.int32).copy()).to(DEV).view(torch.float32)
    t = table(act, 2)
    y, _ = fb.fewbit_fwd(t, x)
    torch.cuda.synchronize()
    s, _ = t.arrays()
    xn, yn = np_bits(x), np_bits(y)
    shards = [wl.shard_range(xn.size, r, _THREADS, 1024) for r in range(_THREADS)]
    y_ref = np.concatenate(list(_POOL.map(lambda c: oracle.fwd(act, 2, s, xn[c[0]:c[1]])[0], shards)))
    d = ulp_distance(yn, y_ref)
    assert d.max() <= 2, (act, int(d.max()), hex(int(bits_all[int(d.argmax())])))
    per_group = stretch + scattered
    in_stretch = (np.arange(xn.size) % per_group) < stretch
    ds = d[in_stretch]
    host_hist = [int((ds == k).sum()) for k in range(3)] + [int((ds > 2).sum())]
    scan_hist = [0, 0, 0, 0]
    for first in firsts:
        r = fb.fewbit_f32_activation_scan(act, first, stretch)
        scan_hist = [a + b for a, b in zip(scan_hist, r["hist"])]
    assert scan_hist == host_hist, (act, scan_hist, host_hist)
