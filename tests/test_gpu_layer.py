"""Parity of qlora_fwd / qlora_bwd_input / qlora_bwd_lora with the CPU oracle on seeded inputs (needs a B200).

Gate: max relative error 2e-2 per output tensor (helpers.rel_err), bf16 inputs and fp32 accumulation on the GPU."""
import numpy as np
import pytest
import torch

import qlora_inputs as qi
from oracle import qlora_oracle as orc
from gpu_util import GpuLayer, to_f64
from helpers import REL_TOL, rel_err

pytestmark = pytest.mark.gpu


def check_layer(layer, rows=None, tol=REL_TOL, **run_kw):
    gl = GpuLayer(layer)
    out = gl.run(**run_kw)
    ref = orc.layer_reference(layer, rows=rows)
    sel = slice(None) if rows is None else np.asarray(rows)
    errs = {"Y": rel_err(to_f64(out["Y"])[sel], ref["Y"]), "dX": rel_err(to_f64(out["dX"])[sel], ref["dX"])}
    if layer["r"]:
        errs["dA"] = rel_err(to_f64(out["dA"]), ref["dA"])
        errs["dB"] = rel_err(to_f64(out["dB"]), ref["dB"])
        if out["H"] is not None:
            errs["H"] = rel_err(to_f64(out["H"])[sel], ref["H"])
            errs["G"] = rel_err(to_f64(out["G"])[sel], ref["G"])
    for name, e in errs.items():
        assert e <= tol, (name, e, errs)
    # the packed matrix produced by the library equals the oracle's
    assert np.array_equal(gl.Q.cpu().numpy(), ref["Q"])
    return errs, out, gl


def sample_rows(M, n=48, seed=0):
    if M <= n:
        return None
    rng = np.random.default_rng(seed)
    rows = set(rng.choice(M, size=n - 4, replace=False).tolist()) | {0, 1, M - 2, M - 1}
    return sorted(rows)


def test_config1_full():
    errs, _, _ = check_layer(qi.config1())
    assert errs["Y"] < 1e-2 and errs["dX"] < 1e-2   # expected a few 2^-9; larger would point at a bug


def test_config2_q_proj_int4():
    check_layer(qi.config2())


def test_config2_as_a_replayed_cuda_graph():
    """The launch configuration the benchmark times: the three calls of several steps captured in one CUDA graph
    (programmatic dependent launches, the pair kernel's self-zeroing counters) and replayed twice; every replay's
    outputs are checked against the oracle on sampled rows and are bitwise those of the call-by-call run."""
    layer = qi.config2(seed=3)
    rows = sample_rows(layer["M"], seed=5)
    _, eager, gl = check_layer(layer, rows=rows)
    import paper_2306_08162_b200 as ql
    M, dev = gl.M, gl.X.device
    bufs = [dict(Y=torch.empty((M, gl.N), dtype=torch.bfloat16, device=dev), dX=torch.empty((M, gl.K), dtype=torch.bfloat16, device=dev),
                 H=torch.empty((M, gl.r), dtype=torch.float32, device=dev), G=torch.empty((M, gl.r), dtype=torch.float32, device=dev),
                 dA=torch.empty((gl.r, gl.K), dtype=torch.float32, device=dev), dB=torch.empty((gl.N, gl.r), dtype=torch.float32, device=dev))
            for _ in range(3)]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for b in bufs:
                ql.qlora_fwd(gl.desc, M, gl.X, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, b["Y"], b["H"], gl.ws)
                ql.qlora_bwd_input(gl.desc, M, gl.dY, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, b["dX"], b["G"], gl.ws)
                ql.qlora_bwd_lora(gl.desc, M, gl.X, gl.dY, gl.A, gl.B, b["H"], b["G"], b["dA"], b["dB"], 0, gl.ws)
    ref = orc.layer_reference(layer, rows=rows)
    sel = np.asarray(rows)
    bits = lambda t: t.view(torch.int16) if t.dtype == torch.bfloat16 else t
    for replay in range(2):
        for b in bufs:
            for t in b.values():
                t.view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32).fill_(-1)      # NaN patterns: nothing is left over
        graph.replay()
        torch.cuda.synchronize()
        assert ql.qlora_device_status() == 0
        for b in bufs:
            assert rel_err(to_f64(b["Y"])[sel], ref["Y"]) <= REL_TOL and rel_err(to_f64(b["dX"])[sel], ref["dX"]) <= REL_TOL
            assert rel_err(to_f64(b["dA"]), ref["dA"]) <= REL_TOL and rel_err(to_f64(b["dB"]), ref["dB"]) <= REL_TOL
            for k in ("Y", "dX", "H", "G", "dA", "dB"):
                assert torch.equal(bits(b[k]), bits(eager[k])), (replay, k)


@pytest.mark.parametrize("which", ["gate", "up", "down"])
def test_config3_mlp_int2_outliers(which):
    layer = qi.config3(which)
    check_layer(layer, rows=sample_rows(layer["M"], seed=1))


@pytest.mark.parametrize("bits", [3, 8])
@pytest.mark.parametrize("M", qi.CONFIG4_M)
def test_config4_int3_int8_sweep(bits, M):
    layer = qi.config4(bits, M)
    check_layer(layer, rows=sample_rows(M, seed=M))


@pytest.mark.parametrize("M", [1, 16, 17, 127, 129, 300])
@pytest.mark.parametrize("bits,g", [(4, 128), (3, 32), (2, 64), (8, 64)])
def test_edge_token_counts(M, bits, g):
    check_layer(qi.random_codes_layer(K=256, N=264, bits=bits, group_size=g, r=8, alpha=16.0, M=M, seed=M + bits))


@pytest.mark.parametrize("K,N", [(11008, 128), (128, 11008), (352, 8), (32, 4096)])
def test_edge_feature_counts(K, N):
    g = 32 if K % 64 else 64
    check_layer(qi.random_codes_layer(K=K, N=N, bits=2, group_size=g, r=16, alpha=32.0, M=40, seed=K + N))


@pytest.mark.parametrize("M", [257, 300, 513, 1000])
@pytest.mark.parametrize("bits,g,K,N", [(4, 128, 256, 320), (2, 64, 320, 256), (3, 64, 512, 192), (8, 128, 384, 576)])
def test_token_counts_above_256_with_ragged_weight_tiles(M, bits, g, K, N):
    """More than 256 tokens selects the CTA-pair kernel (512 tokens x 256 weight rows per tile); K and N here are
    not multiples of 256, so the last weight tile is ragged in both directions, and M leaves a ragged token tile."""
    check_layer(qi.random_codes_layer(K=K, N=N, bits=bits, group_size=g, r=8, alpha=16.0, M=M, seed=M + bits))


@pytest.mark.parametrize("M", [1, 7, 16, 17, 32])
@pytest.mark.parametrize("bits,g,K,N", [(4, 128, 512, 320), (2, 64, 352 * 2, 264), (3, 32, 352, 72), (8, 256, 512, 8), (3, 512, 1024, 4104),
                                        (4, 32, 4128, 40)])
def test_small_token_counts_streaming_kernels(M, bits, g, K, N):
    """Up to 32 tokens go through the TMA-fed streaming kernels: ragged K (not a multiple of the 256-wide stage), ragged N
    (not a multiple of the 32-column CTA tile), every bit width, groups smaller and larger than a stage, more stages
    than ring slots (K = 4128, N = 4104)."""
    check_layer(qi.random_codes_layer(K=K, N=N, bits=bits, group_size=g, r=8, alpha=16.0, M=M, seed=M + bits + K))


@pytest.mark.parametrize("r", [0, 8, 16, 24, 64])
def test_ranks_small_token_counts(r):
    check_layer(qi.random_codes_layer(K=384, N=256, bits=4, group_size=128, r=r, alpha=2.0 * max(r, 1), M=20, seed=40 + r))


@pytest.mark.parametrize("M", [33, 100, 129, 256])
@pytest.mark.parametrize("bits,g,K,N,r", [(4, 128, 1024, 256, 8), (2, 64, 2048, 192, 16), (3, 128, 512, 320, 0), (8, 64, 1536, 128, 64)])
def test_mid_token_counts_split_contraction(M, bits, g, K, N, r):
    """33 .. 256 tokens give few tiles of the single-CTA tensor-core kernel; the contraction is then split over a cluster
    of 2 or 4 CTAs and the parts are added through distributed shared memory (K / 64 steps: 16, 32, 8, 24)."""
    check_layer(qi.random_codes_layer(K=K, N=N, bits=bits, group_size=g, r=r, alpha=2.0 * max(r, 1), M=M, seed=M + bits + r))


@pytest.mark.parametrize("r", [0, 16, 64])
def test_ranks_above_256_tokens(r):
    check_layer(qi.random_codes_layer(K=256, N=512, bits=4, group_size=128, r=r, alpha=2.0 * max(r, 1), M=600, seed=r))


@pytest.mark.parametrize("r", [0, 8, 16, 24, 32, 64])
def test_ranks(r):
    check_layer(qi.random_codes_layer(K=256, N=384, bits=4, group_size=128, r=r, alpha=2.0 * max(r, 1), M=70, seed=r))


def test_group_equals_k_and_small_group():
    check_layer(qi.random_codes_layer(K=512, N=128, bits=4, group_size=512, r=8, alpha=16.0, M=33, seed=1))
    check_layer(qi.random_codes_layer(K=512, N=128, bits=8, group_size=32, r=8, alpha=16.0, M=33, seed=2))


def test_stacked_adapters_through_rank_concatenation():
    """A frozen error-correcting pair (r2 = 32) plus a trainable pair (r = 8) on one quantized layer: run as ONE adapter of
    rank 40 (A rows stacked, the frozen up-projection rescaled by s2 / s, a power of two here, so exact in bf16) and
    checked against the oracle's stacked definition; the trainable pair's gradients are the first 8 rows / columns."""
    K, N, M, r, r2, alpha, alpha2 = 512, 384, 300, 8, 32, 16.0, 16.0
    base = qi.random_codes_layer(K=K, N=N, bits=4, group_size=128, r=r, alpha=alpha, M=M, seed=77)
    A2 = qi.uniform_bf16(78, 1, (r2, K), 1.0 / np.sqrt(K))
    B2 = qi.normal_bf16(78, 2, (N, r2), 0.01)
    s, s2 = alpha / r, alpha2 / r2                                       # 2 and 0.5
    B2_scaled = qi.f32_to_bf16_bits(qi.bf16_bits_to_f32(B2) * np.float32(s2 / s))
    assert np.array_equal(qi.bf16_bits_to_f32(B2_scaled), qi.bf16_bits_to_f32(B2) * np.float32(0.25))   # exact
    cat = dict(base, r=r + r2, alpha=s * (r + r2), A=np.vstack([base["A"], A2]), B=np.hstack([base["B"], B2_scaled]))
    out = GpuLayer(cat).run()
    f64 = orc.bf16_bits_to_f64
    W = orc.dequant(orc.pack(base["codes"], 4), base["scales"], base["zeros"], 4, 128)
    X, dY = f64(base["X"]), f64(base["dY"])
    Y, _ = orc.forward_stacked(X, W, f64(base["A"]), f64(base["B"]), alpha, f64(A2), f64(B2), alpha2)
    dX, dA, dB, _ = orc.backward_stacked(X, dY, W, f64(base["A"]), f64(base["B"]), alpha, f64(A2), f64(B2), alpha2)
    assert rel_err(to_f64(out["Y"]), Y) <= REL_TOL and rel_err(to_f64(out["dX"]), dX) <= REL_TOL
    assert rel_err(to_f64(out["dA"])[:r], dA) <= REL_TOL and rel_err(to_f64(out["dB"])[:, :r], dB) <= REL_TOL


@pytest.mark.parametrize("M,K,N,bits,g,r", [(16, 512, 384, 4, 128, 8), (100, 1024, 256, 2, 64, 16), (600, 512, 512, 4, 128, 8),
                                              (70, 352, 264, 3, 32, 8), (300, 256, 512, 8, 128, 24)])
def test_lora_dropout_against_the_oracle(M, K, N, bits, g, r):
    """LoRA dropout (mask passed in, p = 0.25) through every kernel path: streaming (16 tokens), split single-CTA (100),
    CTA pair (600), CUDA-core fallback (N = 264), rank 24; saved and recomputed H / G."""
    import paper_2306_08162_b200 as ql
    layer = qi.random_codes_layer(K=K, N=N, bits=bits, group_size=g, r=r, alpha=2.0 * r, M=M, seed=900 + M)
    gl = GpuLayer(layer)
    p = 0.25
    mask_np = (np.random.default_rng(M).random((M, K)) >= p).astype(np.uint8)
    mask = torch.from_numpy(mask_np).cuda()
    keep = 1.0 / (1.0 - p)
    Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda"); dX = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    H = torch.empty((M, r), dtype=torch.float32, device="cuda"); G = torch.empty_like(H)
    dA = torch.empty((r, K), dtype=torch.float32, device="cuda"); dB = torch.empty((N, r), dtype=torch.float32, device="cuda")
    ql.qlora_fwd_dropout(gl.desc, M, gl.X, mask, keep, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, Y, H, gl.ws)
    ql.qlora_bwd_input_dropout(gl.desc, M, gl.dY, mask, keep, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, dX, G, gl.ws)
    ql.qlora_bwd_lora_dropout(gl.desc, M, gl.X, mask, keep, gl.dY, gl.A, gl.B, H, G, dA, dB, 0, gl.ws)
    dA2 = torch.empty_like(dA); dB2 = torch.empty_like(dB)
    ql.qlora_bwd_lora_dropout(gl.desc, M, gl.X, mask, keep, gl.dY, gl.A, gl.B, None, None, dA2, dB2, 0, gl.ws)
    torch.cuda.synchronize()
    assert ql.qlora_device_status() == 0
    f64 = orc.bf16_bits_to_f64
    W = orc.dequant(orc.pack(layer["codes"], bits), layer["scales"], layer["zeros"], bits, g)
    Xr, dYr, Ar, Br = f64(layer["X"]), f64(layer["dY"]), f64(layer["A"]), f64(layer["B"])
    Yo, Ho = orc.forward_dropout(Xr, W, Ar, Br, layer["alpha"], mask_np, p)
    dXo, dAo, dBo, Go = orc.backward_dropout(Xr, dYr, W, Ar, Br, layer["alpha"], mask_np, p)
    for name, got, want in (("Y", Y, Yo), ("H", H, Ho), ("dX", dX, dXo), ("G", G, Go), ("dA", dA, dAo), ("dB", dB, dBo)):
        assert rel_err(to_f64(got), want) <= REL_TOL, name
    assert torch.equal(dA, dA2) and torch.equal(dB, dB2)


@pytest.mark.parametrize("M", [20, 400])
def test_activation_order_through_row_permutation_and_column_gather(M):
    """GPTQ activation order: group of feature k = g_idx[k], scattered.  The library runs it as a contiguous-group layer:
    code rows permuted once by a stable sort of g_idx, activation and adapter columns gathered with the same permutation
    (qlora_gather_columns), dX and dA un-permuted with the inverse.  Checked against the oracle evaluated with g_idx."""
    import paper_2306_08162_b200 as ql
    K, N, bits, g, r, alpha = 512, 384, 4, 128, 8, 16.0
    layer = qi.random_codes_layer(K=K, N=N, bits=bits, group_size=g, r=r, alpha=alpha, M=M, seed=300 + M)
    rng = np.random.default_rng(M)
    g_idx = rng.permutation(np.arange(K) // g)
    perm = np.argsort(g_idx, kind="stable").astype(np.int32)
    inv = np.argsort(perm).astype(np.int32)
    f64 = orc.bf16_bits_to_f64
    W = orc.dequant_gidx(orc.pack(layer["codes"], bits), layer["scales"], layer["zeros"], bits, g_idx)
    Xr, dYr, Ar, Br = f64(layer["X"]), f64(layer["dY"]), f64(layer["A"]), f64(layer["B"])
    Yo, _ = orc.forward(Xr, W, Ar, Br, alpha)
    dXo, dAo, dBo, _ = orc.backward(Xr, dYr, W, Ar, Br, alpha)
    # device side: permuted layer
    gl = GpuLayer(dict(layer, codes=np.ascontiguousarray(layer["codes"][perm])))
    d_perm, d_inv = torch.from_numpy(perm).cuda(), torch.from_numpy(inv).cuda()
    Xp, Ap = torch.empty_like(gl.X), torch.empty_like(gl.A)
    ql.qlora_gather_columns(gl.X, d_perm, Xp)
    ql.qlora_gather_columns(gl.A, d_perm, Ap)
    gl.A = Ap
    out = gl.run(X=Xp)
    dX, dA = torch.empty_like(out["dX"]), torch.empty_like(out["dA"])
    ql.qlora_gather_columns(out["dX"].contiguous(), d_inv, dX)
    ql.qlora_gather_columns(out["dA"], d_inv, dA)
    torch.cuda.synchronize()
    assert torch.equal(Xp.cpu(), gl.X.cpu()[:, torch.from_numpy(perm.astype(np.int64))])          # the gather itself is exact
    assert rel_err(to_f64(out["Y"]), Yo) <= REL_TOL and rel_err(to_f64(dX), dXo) <= REL_TOL
    assert rel_err(to_f64(dA), dAo) <= REL_TOL and rel_err(to_f64(out["dB"]), dBo) <= REL_TOL


def test_down_projection_beside_the_tiles_repeats_bitwise_and_on_two_streams():
    """Above 256 tokens with few tiles the pair kernel's spare SM pairs compute H / G during the main loop and publish them
    through a counter pair that the launch zeroes again: repeated launches, and launches of two layers (two workspaces)
    overlapping on two streams, give the same bits as a first, serial run."""
    la = qi.random_codes_layer(K=512, N=512, bits=4, group_size=128, r=8, alpha=16.0, M=600, seed=11)
    lb = qi.random_codes_layer(K=768, N=256, bits=2, group_size=64, r=16, alpha=32.0, M=1000, seed=12)
    _, ra, ga = check_layer(la)
    _, rb, gb = check_layer(lb)
    keys = ("Y", "dX", "H", "G", "dA", "dB")
    bits = lambda t: t.view(torch.int16) if t.dtype == torch.bfloat16 else t
    for _ in range(3):
        again = ga.run()
        for k in keys:
            assert torch.equal(bits(again[k]), bits(ra[k])), k
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    outs = []
    for _ in range(6):
        with torch.cuda.stream(sa):
            Ya = torch.empty_like(ra["Y"]); Ha = torch.empty_like(ra["H"])
            ql_fwd(ga, Ya, Ha)
        with torch.cuda.stream(sb):
            Yb = torch.empty_like(rb["Y"]); Hb = torch.empty_like(rb["H"])
            ql_fwd(gb, Yb, Hb)
        outs.append((Ya, Ha, Yb, Hb))
    torch.cuda.synchronize()
    import paper_2306_08162_b200 as ql
    assert ql.qlora_device_status() == 0
    for Ya, Ha, Yb, Hb in outs:
        assert torch.equal(bits(Ya), bits(ra["Y"])) and torch.equal(Ha, ra["H"])
        assert torch.equal(bits(Yb), bits(rb["Y"])) and torch.equal(Hb, rb["H"])


def ql_fwd(gl, Y, H):
    import paper_2306_08162_b200 as ql
    ql.qlora_fwd(gl.desc, gl.M, gl.X, gl.Q, gl.scales, gl.zeros, gl.A, gl.B, Y, H, gl.ws)


def test_recompute_h_g_matches_saved():
    layer = qi.random_codes_layer(K=512, N=256, bits=4, group_size=128, r=8, alpha=16.0, M=200, seed=3)
    _, saved, gl = check_layer(layer, save_hg=True)
    recomputed = gl.run(save_hg=False)
    assert torch.equal(saved["dA"], recomputed["dA"]) and torch.equal(saved["dB"], recomputed["dB"])


@pytest.mark.parametrize("M,K,N,r", [(600, 512, 512, 8), (1000, 2112, 320, 16), (300, 1024, 11008, 8), (1024, 256, 10240, 8)])
def test_down_projection_has_the_same_bits_inside_the_kernel_and_as_a_launch(M, K, N, r):
    """Above 256 tokens H / G come from the tensor-core kernel's producer clusters when its tiles leave SM pairs idle and
    from a stand-alone launch otherwise (here: the recomputation inside qlora_bwd_lora).  The streaming code sums in an
    order that depends on the contraction length only, so saved and recomputed H / G give bitwise the same gradients.
    (Last case: 80 forward tiles on 74 pairs, so the producers are pairs with one tile fewer that take tiles afterwards.)"""
    layer = qi.random_codes_layer(K=K, N=N, bits=4, group_size=64, r=r, alpha=2.0 * r, M=M, seed=17)
    _, saved, gl = check_layer(layer, save_hg=True)
    recomputed = gl.run(save_hg=False)
    assert torch.equal(saved["dA"], recomputed["dA"]) and torch.equal(saved["dB"], recomputed["dB"])


def test_many_tokens_narrow_layer():
    """20000 tokens through a narrow layer: 40 token tiles of the pair kernel on a single column tile, and a down-projection
    launch with more 16-row blocks (1250) than one wave of CTAs holds (148 x 8), so its grid goes over several waves."""
    layer = qi.random_codes_layer(K=256, N=128, bits=4, group_size=64, r=8, alpha=16.0, M=20000, seed=23)
    check_layer(layer)


@pytest.mark.parametrize("seed", range(24))
def test_seeded_sweep_across_the_dispatch_boundaries(seed):
    """Seeded random shapes around every switch of the dispatch (16 / 17, 32 / 33, 256 / 257, the cost-model range up to
    1024, above it), all bit widths, ranks fused and not: each against the oracle."""
    rng = np.random.default_rng(1234 + seed)
    M = int(rng.choice([1, 9, 16, 17, 31, 32, 33, 100, 256, 257, 300, 512, 513, 700, 769, 1000, 1024, 1025, 1300]))
    bits = int(rng.choice([2, 3, 4, 8]))
    g = int(rng.choice([64, 128]))
    K = int(rng.choice([128, 256, 384, 640, 1024, 2176]))
    N = int(rng.choice([64, 128, 320, 704, 1536, 2752]))
    r = int(rng.choice([0, 8, 16, 24]))
    layer = qi.random_codes_layer(K=K, N=N, bits=bits, group_size=g, r=r, alpha=2.0 * max(r, 8), M=M, seed=100 + seed)
    check_layer(layer)


def test_accumulate_adds_to_existing_gradients():
    layer = qi.random_codes_layer(K=256, N=256, bits=4, group_size=128, r=8, alpha=16.0, M=96, seed=4)
    gl = GpuLayer(layer)
    first = gl.run()
    dA0 = torch.full_like(first["dA"], 3.0)
    dB0 = torch.full_like(first["dB"], -2.0)
    second = gl.run(accumulate=1, dA=dA0.clone(), dB=dB0.clone())
    assert torch.equal(second["dA"], dA0 + first["dA"]) and torch.equal(second["dB"], dB0 + first["dB"])


def test_bitwise_deterministic():
    layer = qi.config1(seed=2)
    gl = GpuLayer(layer)
    a = gl.run()
    b = gl.run()
    for k in ("Y", "dX", "dA", "dB"):
        assert torch.equal(a[k].view(torch.int16) if a[k].dtype == torch.bfloat16 else a[k],
                           b[k].view(torch.int16) if b[k].dtype == torch.bfloat16 else b[k]), k


def test_b_zero_gives_pure_quantized_layer():
    layer = qi.random_codes_layer(K=256, N=128, bits=4, group_size=128, r=8, alpha=16.0, M=64, seed=5)
    layer["B"] = np.zeros_like(layer["B"])
    errs, out, gl = check_layer(layer)
    W = orc.dequant(orc.pack(layer["codes"], 4), layer["scales"], layer["zeros"], 4, 128)
    X = orc.bf16_bits_to_f64(layer["X"])
    assert rel_err(to_f64(out["Y"]), X @ W.T) <= REL_TOL
    assert float(out["dA"].abs().max()) == 0.0


def test_empty_batch_is_a_no_op():
    layer = qi.random_codes_layer(K=64, N=64, bits=4, group_size=32, r=8, alpha=16.0, M=4, seed=6)
    gl = GpuLayer(layer)
    out = gl.run(X=gl.X[:0], dY=gl.dY[:0], check_canaries=True)
    assert float(out["dA"].abs().max()) == 0.0 and float(out["dB"].abs().max()) == 0.0


@pytest.mark.parametrize("K,N,M,bits,g,r", [(1024, 6656, 1536, 4, 128, 8), (6656, 1024, 1536, 2, 64, 16),
                                            (1024, 6656, 1400, 3, 128, 8), (1024, 6656, 1536, 8, 128, 0)])
def test_last_wave_split_along_the_contraction(K, N, M, bits, g, r):
    """78 tiles of 512 tokens x 256 weight rows on 74 SM pairs: the four left-over tiles are each shared by two pairs,
    half of the contraction each, which exchange halves of the result through the workspace (forward for N = 6656,
    backward for K = 6656).  Parity on sampled rows of every token tile, and the same bits on a second run."""
    layer = qi.random_codes_layer(K=K, N=N, bits=bits, group_size=g, r=r, alpha=16.0, M=M, seed=K // 64 + bits)
    rows = sorted(set(sample_rows(M, n=60, seed=3)) | {511, 512, 1023, 1024})
    _, out, gl = check_layer(layer, rows=rows)
    again = gl.run()
    for key in ("Y", "dX"):
        assert torch.equal(out[key].view(torch.int16), again[key].view(torch.int16)), key
