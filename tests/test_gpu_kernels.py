"""Kernel-level parity on the GPU, each entry point called through the C ABI and
compared element by element with the CPU oracle (or, for a plain matrix product,
with its definition in float64)."""
import numpy as np
import pytest

from oracle import dllm_oracle as O
from paper_2506_06295_b200 import synth
from tests.helpers import rel_l2, selection_matches

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2506_06295_b200 import build as build_mod
    build_mod.build()
    from paper_2506_06295_b200 import dllm
    assert torch.cuda.is_available()
    return torch, dllm


GEMM_SHAPES = [
    (4400, 384, 128),    # 18 activation tiles: the launch-order remap with a narrow last group (16 + 2)
    (3, 200, 320),       # tiny M (long-prompt regime), ragged N
    (64, 4096, 4096),    # selected rows x a square projection: split-K
    (70, 1536, 832),     # ragged M, K = 13 blocks
    (130, 640, 448),     # M tail of 2 in a 256 tile
    (256, 512, 3584),    # GQA V projection shape: few N tiles
    (600, 384, 128),     # several M tiles, two k blocks
    (64, 24576, 512),    # many N tiles: no split
]


@pytest.mark.parametrize("M,N,K", GEMM_SHAPES)
def test_gemm_bf16_tcgen05(env, M, N, K):
    torch, dllm = env
    A = synth.round_to_bf16(synth.random_normal((M, K), seed=M + K))
    W = synth.round_to_bf16(synth.random_normal((N, K), seed=N + 7 * K, std=0.05))
    dA = torch.from_numpy(A).cuda().to(torch.bfloat16)
    dW = torch.from_numpy(W).cuda().to(torch.bfloat16)
    got = dllm.gemm_bf16(dA, dW).cpu().numpy()
    want = A.astype(np.float64) @ W.astype(np.float64).T
    assert rel_l2(got, want) < 2e-6
    assert np.abs(got - want).max() < 1e-4 * np.abs(want).max()
    # bit-reproducible and independent of the other rows in the launch
    again = dllm.gemm_bf16(dA, dW).cpu().numpy()
    assert np.array_equal(got, again)
    if M > 8:
        sub = dllm.gemm_bf16(dA[: M // 2].contiguous(), dW).cpu().numpy()
        assert rel_l2(sub, want[: M // 2]) < 2e-6


@pytest.mark.parametrize("act_tile,splits,stages", [(32, 1, 2), (64, 3, 4), (128, 2, 3), (128, 5, 6), (256, 1, 4),
                                                    (256, 4, 2), (0, 0, 0), (64, 13, 9)])
def test_gemm_bf16_explicit_plans(env, act_tile, splits, stages):
    """Every activation-tile shape, split factor and ring depth gives the same product; with reduce=False the
    split-K slabs are left in the scratch buffer and add up to it in slab order."""
    torch, dllm = env
    M, N, K = 150, 900, 832          # ragged M and N, 13 k-blocks
    A = synth.round_to_bf16(synth.random_normal((M, K), seed=5))
    W = synth.round_to_bf16(synth.random_normal((N, K), seed=6, std=0.05))
    dA = torch.from_numpy(A).cuda().to(torch.bfloat16)
    dW = torch.from_numpy(W).cuda().to(torch.bfloat16)
    want = A.astype(np.float64) @ W.astype(np.float64).T
    got = dllm.gemm_bf16_planned(dA, dW, act_tile, splits, stages).cpu().numpy()
    assert rel_l2(got, want) < 2e-6
    sb = dllm.lib.dllm_gemm_bf16_planned_scratch_bytes(M, N, K, act_tile, splits)
    if sb:
        scratch = torch.zeros(sb, dtype=torch.uint8, device="cuda")
        dllm.gemm_bf16_planned(dA, dW, act_tile, splits, stages, scratch=scratch, reduce=False)
        slabs = scratch.view(torch.float32).cpu().numpy().reshape(-1, M, N)
        acc = slabs[0].copy()
        for sl in slabs[1:]:
            acc += sl
        assert np.array_equal(acc, got)      # the reduction adds the slabs in index order
    assert dllm.lib.dllm_gemm_bf16_planned(None, None, None, M, N, K, 48, 0, 0, None, 0, None) == dllm.INVALID_ARG


@pytest.mark.parametrize("M,m,K,act_tile", [(64, 1216, 512, 0), (3, 64, 64, 32), (70, 832, 448, 64), (130, 192, 1088, 128),
                                            (300, 320, 256, 256), (257, 128, 832, 0),
                                            (300, 256, 192, 0),      # default plan: CTA pairs, 128-row tiles
                                            (200, 9472, 64, 0),      # default plan: CTA pairs, 256-row tiles
                                            (600, 19200, 64, 0)])    # CTA pairs, 256-row tiles, three row tiles
def test_ffn_gate_up_epilogue(env, M, m, K, act_tile):
    """Gate / up projection with SwiGLU in the GEMM epilogue against silu(A Wg^T) * (A Wu^T) in float64."""
    torch, dllm = env
    A = synth.round_to_bf16(synth.random_normal((M, K), seed=M + 3))
    Wg = synth.round_to_bf16(synth.random_normal((m, K), seed=m + 1, std=0.08))
    Wu = synth.round_to_bf16(synth.random_normal((m, K), seed=m + 2, std=0.08))
    Wgu = np.stack([Wg.reshape(m // 64, 64, K), Wu.reshape(m // 64, 64, K)], axis=1).reshape(2 * m, K)
    dA = torch.from_numpy(A).cuda().to(torch.bfloat16)
    dW = torch.from_numpy(np.ascontiguousarray(Wgu)).cuda().to(torch.bfloat16)
    got = dllm.ffn_gate_up_bf16(dA, dW, act_tile).float().cpu().numpy()
    gate = A.astype(np.float64) @ Wg.astype(np.float64).T
    want = gate / (1 + np.exp(-gate)) * (A.astype(np.float64) @ Wu.astype(np.float64).T)
    assert rel_l2(got, want) < 3e-3                                     # one rounding to bf16: 2^-9 per element
    assert np.abs(got - want).max() <= 2 ** -8 * np.abs(want).max() + 1e-6
    assert np.array_equal(got, dllm.ffn_gate_up_bf16(dA, dW, act_tile).float().cpu().numpy())
    assert dllm.lib.dllm_ffn_gate_up_bf16(None, None, None, M, m, K, 0, 0, None) == dllm.INVALID_ARG
    assert dllm.lib.dllm_ffn_gate_up_bf16(dA.data_ptr(), dW.data_ptr(), dA.data_ptr(), M, 100, K, 0, 0, None) == dllm.INVALID_ARG


@pytest.mark.parametrize("M,N,K,act_tile,splits,stages", [
    (256, 256, 64, 256, 1, 2),        # one pair, one k-block
    (130, 512, 448, 128, 1, 3),       # 128-row tiles, ragged second tile
    (256, 4096, 4096, 256, 4, 3),     # the V projection of a 256-token response
    (300, 768, 832, 256, 3, 5),       # two activation tiles, 13 k-blocks in 3 splits
    (768, 1024, 1024, 256, 0, 0),     # default split and ring depth
    (70, 256, 320, 128, 2, 2),        # fewer rows than a tile
])
def test_gemm_bf16_cta_pairs(env, M, N, K, act_tile, splits, stages):
    """The CTA-pair kernel (cta_group::2) gives the product, bit-identical to the one-CTA kernel with the same
    tile rows and k ranges (the same sums in the same order)."""
    torch, dllm = env
    A = synth.round_to_bf16(synth.random_normal((M, K), seed=M + K + 3))
    W = synth.round_to_bf16(synth.random_normal((N, K), seed=N + 5 * K, std=0.05))
    dA = torch.from_numpy(A).cuda().to(torch.bfloat16)
    dW = torch.from_numpy(W).cuda().to(torch.bfloat16)
    got = dllm.gemm_bf16_pair(dA, dW, act_tile, splits, stages).cpu().numpy()
    want = A.astype(np.float64) @ W.astype(np.float64).T
    assert rel_l2(got, want) < 2e-6
    assert np.array_equal(got, dllm.gemm_bf16_pair(dA, dW, act_tile, splits, stages).cpu().numpy())
    if splits:
        one = dllm.gemm_bf16_planned(dA, dW, act_tile, splits, stages).cpu().numpy()
        assert np.array_equal(got, one)
    assert dllm.lib.dllm_gemm_bf16_pair(dA.data_ptr(), dW.data_ptr(), dA.data_ptr(), M, 128, K, 256, 0, 0, None, 0, None) == dllm.INVALID_ARG


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_gemm_simt(env, dtype):
    torch, dllm = env
    M, N, K = 77, 200, 328
    A = synth.random_normal((M, K), seed=1)
    W = synth.random_normal((N, K), seed=2, std=0.05)
    if dtype == "bf16":
        A, W = synth.round_to_bf16(A), synth.round_to_bf16(W)
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    got = dllm.gemm_simt(torch.from_numpy(A).cuda().to(td), torch.from_numpy(W).cuda().to(td)).cpu().numpy()
    want = A.astype(np.float64) @ W.astype(np.float64).T
    assert rel_l2(got, want) < 2e-6


ATT_CASES = [
    # B, a, n, H, Hkv, hd
    (1, 8, 96, 4, 4, 64),      # tiny configuration, partial step
    (2, 19, 77, 5, 5, 64),     # ragged queries and keys
    (1, 3, 300, 4, 4, 128),    # few queries, longer keys
    (2, 33, 130, 7, 1, 64),    # GQA, 7 query heads per KV head
    (1, 64, 768, 8, 8, 128),   # LLaDA-8B partial-step shape, 8 of the 32 heads
    (1, 128, 512, 28, 4, 128), # Dream-7B partial-step shape
    (1, 3, 4128, 2, 2, 128),   # long-prompt regime: 3 queries, 65 key tiles, ragged last tile (few-rows kernel, 6 ways)
    (2, 30, 1100, 3, 3, 64),   # few-rows kernel with two row groups and 3 ways, 18 key tiles, head_dim 64
    (1, 5, 2000, 8, 2, 128),   # grouped heads: 20 rows per KV head, few-rows kernel, ragged last tile
    (3, 16, 1024, 2, 2, 128),  # exactly 16 rows and 16 key tiles: the smallest shape of the few-rows kernel
    (2, 200, 333, 4, 2, 64),   # several row tiles, G = 2, ragged keys
    # more than 64 (query, head-of-group) rows per KV head: the tcgen05 kernel (two 128-row tiles per CTA, 64-key tiles)
    (1, 256, 768, 8, 8, 128),  # LLaDA-8B response-refresh shape, 8 of the 32 heads
    (1, 130, 1000, 2, 2, 128), # ragged second row tile (2 rows), 16 key tiles with a ragged last one
    (1, 65, 64, 1, 1, 128),    # smallest case of that kernel: one row tile, one key tile
    (3, 90, 260, 6, 2, 64),    # head_dim 64, G = 3, three sequences
    (1, 300, 520, 4, 4, 128),  # two CTAs per head, the second with one live row tile; 9 key tiles: the ring is reused
    (2, 512, 1536, 2, 2, 128), # batched-serving refresh shape: 24 key tiles, two full CTAs per (sequence, head)
    (1, 40, 200, 28, 4, 128),  # grouped heads: 280 rows per KV head gathered from 7 query heads (no TMA for Q)
    (1, 200, 3000, 1, 1, 64),  # head_dim 64, one CTA's worth of rows against 47 key tiles: many key-range splits
    # one live 128-row tile per CTA: its two softmax groups take the even and the odd key tiles and merge at the end
    (1, 100, 1000, 4, 4, 128), # ragged rows, 16 key tiles with a ragged last one
    (2, 128, 520, 2, 2, 64),   # nine key tiles: five for group 0, four for group 1 (the last with 8 keys)
    (1, 128, 512, 2, 2, 128),  # eight key tiles, the fewest that are shared
    (1, 128, 448, 2, 2, 128),  # seven key tiles: not shared, the second group idles
    (4, 128, 1536, 4, 4, 128), # batched adaptive step shape: 24 key tiles per CTA
]


@pytest.mark.parametrize("case", ATT_CASES)
@pytest.mark.parametrize("dtype", ["fp32", "bf16", "bf16_nosplit"])
def test_attention(env, case, dtype):
    torch, dllm = env
    B, a, n, H, Hkv, hd = case
    q = synth.random_normal((B * a, H * hd), seed=11, std=1.3)
    k = synth.random_normal((B, n, Hkv * hd), seed=12, std=1.3)
    v = synth.random_normal((B, n, Hkv * hd), seed=13)
    split = dtype != "bf16_nosplit"
    dtype = dtype[:4]
    if dtype == "bf16":
        q, k, v = (synth.round_to_bf16(t) for t in (q, k, v))
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    got = dllm.attention(*(torch.from_numpy(t).cuda().to(td) for t in (q, k, v)), B, a, n, H, Hkv, hd, split=split)
    got = got.to(torch.float32).cpu().numpy()
    for b in range(B):
        want = O.attention(q[b * a:(b + 1) * a].astype(np.float64).reshape(a, H, hd),
                           k[b].astype(np.float64).reshape(n, Hkv, hd),
                           v[b].astype(np.float64).reshape(n, Hkv, hd), Hkv)
        tol = 1e-5 if dtype == "fp32" else 8e-3       # bf16: output rounding 2^-9 plus P rounded to bf16
        assert rel_l2(got[b * a:(b + 1) * a], want) < tol


@pytest.mark.parametrize("case", [
    (1, 256, 768, 2, 2, 128),   # tcgen05 kernel, two row tiles per CTA, 12 key tiles
    (2, 128, 1024, 2, 2, 128),  # tcgen05 kernel, one row tile shared by the two softmax groups, 16 key tiles
    (1, 200, 640, 3, 1, 64),    # tcgen05 kernel, head_dim 64, grouped heads
    (1, 64, 768, 2, 2, 128),    # 64-row mma.sync kernel
    (1, 3, 2048, 2, 2, 128),    # few-rows kernel
])
@pytest.mark.parametrize("split", [True, False])
def test_attention_with_row_maxima_that_keep_growing(env, case, split):
    """Keys whose norm grows with their index: every later key tile raises the running maxima of the online
    softmax by many powers of two, so the accumulated output and sum are rescaled again and again (the lazy
    rescale of the tcgen05 kernel only acts beyond 2^8).  Eq. for attention as in Sec. A.7; the oracle is exact."""
    torch, dllm = env
    B, a, n, H, Hkv, hd = case
    q = synth.random_normal((B * a, H * hd), seed=21, std=8.0)
    ramp = np.linspace(0.15, 1.0, n, dtype=np.float32)[None, :, None]
    k = synth.random_normal((B, n, Hkv * hd), seed=22, std=1.3) * ramp
    v = synth.random_normal((B, n, Hkv * hd), seed=23)
    q, k, v = (synth.round_to_bf16(t) for t in (q, k, v))
    got = dllm.attention(*(torch.from_numpy(t).cuda().to(torch.bfloat16) for t in (q, k, v)), B, a, n, H, Hkv, hd,
                         split=split)
    got = got.to(torch.float32).cpu().numpy()
    assert np.isfinite(got).all()
    for b in range(B):
        want = O.attention(q[b * a:(b + 1) * a].astype(np.float64).reshape(a, H, hd),
                           k[b].astype(np.float64).reshape(n, Hkv, hd),
                           v[b].astype(np.float64).reshape(n, Hkv, hd), Hkv)
        assert rel_l2(got[b * a:(b + 1) * a], want) < 8e-3


@pytest.mark.parametrize("M,N,K", [(520, 7680, 320), (4400, 1280, 200), (300, 20000, 64)])
def test_gemm_persistent_kernel_is_bit_identical_to_the_one_tile_kernel(env, M, N, K):
    """Unsplit products with more tiles than SMs run on the persistent kernel (one CTA per SM walks through the
    tiles, two accumulators, epilogue under the next main loop).  Same k loop per tile: the same bits as the
    one-tile-per-CTA kernel, for the plain epilogue and for the SwiGLU epilogue; ragged activation tiles, a ragged
    k block, more than 16 activation tiles (the launch-order remap), fewer tiles than SMs."""
    torch, dllm = env
    A = torch.from_numpy(synth.round_to_bf16(synth.random_normal((M, K), seed=21))).cuda().to(torch.bfloat16)
    W = torch.from_numpy(synth.round_to_bf16(synth.random_normal((N, K), seed=22, std=0.05))).cuda().to(torch.bfloat16)
    out = {}
    try:
        for mode in (-1, 1):
            dllm._check(dllm.lib.dllm_debug_gemm_plan(mode))
            c = dllm.gemm_bf16_planned(A, W, act_tile=256, splits=1)
            g = dllm.ffn_gate_up_bf16(A, W[:N // 128 * 128], act_tile=256) if K % 8 == 0 else None
            torch.cuda.synchronize()
            out[mode] = (c.cpu().numpy(), g.float().cpu().numpy())
    finally:
        dllm._check(dllm.lib.dllm_debug_gemm_plan(0))
    dllm.kernel_status()
    want = A.double().cpu().numpy() @ W.double().cpu().numpy().T
    assert rel_l2(out[1][0], want) < 1e-5
    assert np.array_equal(out[-1][0], out[1][0])
    assert np.array_equal(out[-1][1], out[1][1])


@pytest.mark.parametrize("M,N,K,forced", [(576, 20000, 320, 0), (530, 1280, 200, 192), (192, 384, 64, 192)])
def test_gemm_192_row_tiles(env, M, N, K, forced):
    """Activation tiles of 192 rows in the persistent kernel (the 576 rows of a mixed step are 3 x 192, not
    3 x 256): the default plan takes them for 576 rows against many weight tiles; ragged last tile, a ragged k
    block, a single tile.  The k loop per output element is the same: the same bits as with 256-row tiles, for
    the plain and for the SwiGLU epilogue."""
    torch, dllm = env
    A = torch.from_numpy(synth.round_to_bf16(synth.random_normal((M, K), seed=31))).cuda().to(torch.bfloat16)
    W = torch.from_numpy(synth.round_to_bf16(synth.random_normal((N, K), seed=32, std=0.05))).cuda().to(torch.bfloat16)
    Wg = W[:N // 128 * 128]
    c = dllm.gemm_bf16_planned(A, W, act_tile=forced, splits=1).cpu().numpy()
    g = dllm.ffn_gate_up_bf16(A, Wg, act_tile=forced).float().cpu().numpy()
    c256 = dllm.gemm_bf16_planned(A, W, act_tile=256, splits=1).cpu().numpy()
    g256 = dllm.ffn_gate_up_bf16(A, Wg, act_tile=256).float().cpu().numpy()
    dllm.kernel_status()
    want = A.double().cpu().numpy() @ W.double().cpu().numpy().T
    assert rel_l2(c, want) < 1e-5
    assert np.array_equal(c, c256) and np.array_equal(g, g256)
    assert dllm.lib.dllm_gemm_bf16_planned(A.data_ptr(), W.data_ptr(), A.data_ptr(), M, N, K, 192, 2, 0, None, 0, None) == dllm.INVALID_ARG


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("B,R,width,k", [(1, 32, 256, 8), (3, 256, 4096, 64), (2, 100, 512, 50), (1, 512, 4096, 51),
                                         # the longest response the selection kernel admits (keys and flags of one
                                         # sequence in more than 48 KB of shared memory) and one just past that mark
                                         (1, 8192, 64, 819), (2, 6000, 64, 1500)])
def test_vverify_select(env, dtype, B, R, width, k):
    torch, dllm = env
    cache = synth.random_normal((B, R, width), seed=5)
    noise = synth.random_normal((B, R, width), seed=6)
    amp = synth.random_uniform((B, R, 1), seed=7) ** 4            # most rows barely move, a few move a lot
    new = cache + amp * noise
    new[:, ::3] = cache[:, ::3]                                     # a third of the rows are exactly unchanged
    if dtype == "bf16":
        cache, new = synth.round_to_bf16(cache), synth.round_to_bf16(new)
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    d_new = torch.from_numpy(new).cuda().to(td)
    d_cache = torch.from_numpy(cache).cuda().to(td)
    sim, idx = dllm.vverify_select(d_new, d_cache, k)
    torch.cuda.synchronize()
    sim, idx = sim.cpu().numpy(), idx.cpu().numpy()
    assert torch.equal(d_cache, d_new)                              # whole V overwritten
    for b in range(B):
        s = O.cosine_rows(new[b].astype(np.float64), cache[b].astype(np.float64))
        np.testing.assert_allclose(sim[b], s, atol=2e-6)
        assert (sim[b, ::3] == 1.0).all()                           # unchanged rows give exactly 1
        want = O.select_lowest(s, k)
        assert list(idx[b]) == sorted(idx[b]) and len(set(idx[b].tolist())) == k
        assert selection_matches(idx[b], want, s)
        # the kernel's own similarities, sorted by the same key, must give exactly its set
        keys = sorted((int(np.rint(float(sim[b, j]) * 2 ** 20)), j) for j in range(R))
        assert idx[b].tolist() == sorted(j for _, j in keys[:k])
