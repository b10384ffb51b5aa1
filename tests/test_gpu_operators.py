"""Operator-level GPU parity (need a B200): the stand-alone tree-attention and small-M GEMM entry points of
the C ABI against the CPU oracle, plus the bitwise row-invariance the lossless guarantee rests on."""
import numpy as np
import pytest
import torch

import synth
import paper_2603_17942_b200 as P
from oracle import esp as O

pytestmark = pytest.mark.gpu

R = P.ESP_MAX_ROWS


# ------------------------------------------------------------------ small-M GEMM
def _gemm(impl, x, w, rows):
    n_out, k_in = w.shape
    xd = torch.zeros(R, k_in, dtype=torch.bfloat16, device="cuda")
    xd[:rows] = x.cuda()
    y = torch.full((R, n_out), float("nan"), dtype=torch.float32, device="cuda")
    nb = P.esp_gemm_scratch_bytes()
    scratch = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    P.esp_gemm_bf16(impl, rows, n_out, k_in, xd, w, y, scratch, nb)
    torch.cuda.synchronize()
    return y[:rows].cpu().numpy()


@pytest.mark.parametrize("rows,n_out,k_in", [(1, 128, 64), (68, 384, 512), (80, 1000, 688), (68, 6144, 4096),
                                             (5, 4096, 14336), (68, 20000, 4096)])
def test_gemm_bf16_against_oracle(rows, n_out, k_in):
    """y = x W^T for bf16 operands with fp32 accumulation.  Products of bf16 values are exact in fp32, so the
    only difference to the oracle's running sum is the order of the fp32 additions."""
    g = torch.Generator().manual_seed(rows * 7919 + n_out)
    x = torch.randn(rows, k_in, generator=g).bfloat16()
    w = (torch.randn(n_out, k_in, generator=g) * 0.05).bfloat16().cuda()
    ref = O.linear(x.float().numpy(), w.cpu())
    scale = np.abs(ref).max()
    for impl in (0, 1):
        got = _gemm(impl, x, w, rows)
        assert np.isfinite(got).all()
        assert np.abs(got - ref).max() <= 2e-5 * scale, f"impl {impl}"


def test_gemm_rows_do_not_depend_on_their_neighbours():
    """A row's result has the same bits whether it runs alone or among 79 others (the tensor-core kernel is
    launched with one fixed tile shape and one fixed k split for every row count)."""
    g = torch.Generator().manual_seed(5)
    k_in, n_out = 4096, 4096
    x = torch.randn(R, k_in, generator=g).bfloat16()
    w = (torch.randn(n_out, k_in, generator=g) * 0.05).bfloat16().cuda()
    full = _gemm(0, x, w, R)
    for r in (0, 37, 79):
        alone = _gemm(0, x[r:r + 1], w, 1)
        assert np.array_equal(alone[0], full[r])
    again = _gemm(0, x, w, R)
    assert np.array_equal(full, again)       # run-to-run deterministic (no arrival-order dependence)


# ------------------------------------------------------------------ tree attention (the stand-alone operator workload)
def _tree_block(n_nodes, n_probes, max_depth, seed):
    parents = synth.random_tree_parents(n_nodes, max_depth, seed)
    M = n_nodes + n_probes
    depth = np.zeros(M, np.int32)
    vis = np.zeros((M, M), np.uint8)
    for i in range(n_nodes):
        a = i
        while a >= 0:
            vis[i, a] = 1
            a = int(parents[a])
        depth[i] = vis[i].sum() - 1
    for j in range(n_probes):        # a mask-probe chain under the root
        r = n_nodes + j
        vis[r, 0] = 1
        vis[r, n_nodes:r + 1] = 1
        depth[r] = j + 1
    return parents, depth, vis


def _anc_words(vis):
    M = vis.shape[0]
    anc = np.zeros((R, 2), np.uint64)
    for r in range(M):
        for i in range(M):
            if vis[r, i]:
                anc[r, i // 64] |= np.uint64(1) << np.uint64(i % 64)
    for r in range(M, R):
        anc[r, r // 64] = np.uint64(1) << np.uint64(r % 64)
    return anc


def _run_attention(dtype, q, kc, vc, anc, depth, n_rows, L, Hq, Hkv, h, dcap=16):
    """q [b,R,Hq,h]; kc/vc [b,Hkv,cap,h] with block rows already at L+i; anc [b,R,2]; depth [b,R]."""
    b, cap = kc.shape[0], kc.shape[2]
    out = torch.zeros_like(q)
    nb = P.esp_tree_attention_scratch_bytes(b, Hq, h, cap)
    scratch = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    P.esp_tree_attention(dtype, b, n_rows, L, cap, Hq, Hkv, h, dcap, q, kc, vc,
                         torch.from_numpy(anc.view(np.int64)).cuda(), torch.from_numpy(depth).cuda(), out, scratch, nb)
    torch.cuda.synchronize()
    assert P.esp_tree_attention_status(scratch) == 0       # no bounded wait ran out, no index left its range
    return out


def test_tree_attention_status_reports_a_set_error_word():
    """The operator reports device-side problems through the first word of its scratch.  The read-back is checked
    from the host side: a word set by hand must come back as ESP_E_DEVICE, and the next call must clear it."""
    Hq, Hkv, h, L = 32, 8, 128, 300
    cap = L + R
    q, kc, vc, _, _ = synth.random_qkv((1, R, Hq, h), (1, Hkv, cap, h), (1, Hkv, 4, h), seed=1, device="cuda")
    anc = np.zeros((1, R, 2), np.uint64)
    for i in range(R):
        anc[0, i, i // 64] = np.uint64(1) << np.uint64(i % 64)
    nb = P.esp_tree_attention_scratch_bytes(1, Hq, h, cap)
    scratch = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    args = (1, 1, 4, L, cap, Hq, Hkv, h, 16, q, kc, vc, torch.from_numpy(anc.view(np.int64)).cuda(),
            torch.zeros((1, R), dtype=torch.int32, device="cuda"), torch.zeros_like(q), scratch, nb)
    P.esp_tree_attention(*args)
    assert P.esp_tree_attention_status(scratch) == 0
    scratch[:4] = torch.tensor([2, 0, 0, 0], dtype=torch.uint8, device="cuda")     # as a kernel would record DEV_E_INDEX
    with pytest.raises(P.EspError) as e:
        P.esp_tree_attention_status(scratch)
    assert e.value.code == -5                               # ESP_E_DEVICE
    P.esp_tree_attention(*args)
    assert P.esp_tree_attention_status(scratch) == 0


@pytest.mark.parametrize("batch,L,dt", [(1, 4096, "bf16"), (16, 4096, "bf16"), (4, 4096, "bf16"), (2, 777, "bf16"),
                                        (1, 0, "bf16"), (1, 5, "bf16"), (2, 300, "fp32")])
def test_tree_attention_against_oracle(batch, L, dt):
    """32 query heads / 8 KV heads of 128, N(0,1) cache, a 64-node random tree of depth <= 5 plus 4 mask-probe
    rows.  The split length follows the batch: 16 splits of 256 positions for one sequence at 4096, one split of
    4096 for 16 sequences, 4 splits of 1024 for 4 sequences (items of 8 chunks on the persistent kernel, merged
    over splits).  Tolerance: the output is a convex combination of N(0,1) values, bf16 rounding of the probabilities
    and of the output bounds the error by a few 2^-8 relative steps; 2e-2 absolute covers it."""
    Hq, Hkv, h, n_nodes, n_probes = 32, 8, 128, 64, 4
    M = n_nodes + n_probes
    cap = L + R
    tdt = torch.bfloat16 if dt == "bf16" else torch.float32
    q, kc, vc, kb, vb = synth.random_qkv((batch, R, Hq, h), (batch, Hkv, cap, h), (batch, Hkv, M, h), seed=L + batch,
                                         device="cuda", dtype=tdt)
    kc[:, :, L:L + M] = kb
    vc[:, :, L:L + M] = vb
    anc = np.zeros((batch, R, 2), np.uint64)
    depth = np.zeros((batch, R), np.int32)
    vis_all = []
    for s in range(batch):
        _, d, vis = _tree_block(n_nodes, n_probes, 5, seed=100 * L + s)
        anc[s] = _anc_words(vis)
        depth[s, :M] = d
        vis_all.append(vis)
    out = _run_attention(0 if dt == "fp32" else 1, q, kc, vc, anc, depth, M, L, Hq, Hkv, h)
    tol = 2e-2 if dt == "bf16" else 2e-5
    for s in sorted({0, batch // 2, batch - 1}):
        ref = O.tree_attention(q[s, :M].float().cpu().numpy(), kc[s, :, :L].float().permute(1, 0, 2).cpu().numpy(),
                               vc[s, :, :L].float().permute(1, 0, 2).cpu().numpy(),
                               kb[s].float().permute(1, 0, 2).cpu().numpy(), vb[s].float().permute(1, 0, 2).cpu().numpy(),
                               vis_all[s])
        got = out[s, :M].float().cpu().numpy()
        assert np.isfinite(got).all()
        assert np.abs(got - ref).max() <= tol, f"sequence {s}"


def test_tree_attention_rows_equal_decoding_each_path_alone():
    """Bitwise: a node verified inside the tree block gets the bits it would get if its ancestors had been
    accepted into the cache and it were decoded alone (what lossless verification needs)."""
    Hq, Hkv, h, n_nodes, n_probes, L = 32, 8, 128, 64, 4, 1500
    M = n_nodes + n_probes
    cap = L + R + 16                                  # room for the deepest path moved into the cache
    q, kc, vc, kb, vb = synth.random_qkv((1, R, Hq, h), (1, Hkv, cap, h), (1, Hkv, M, h), seed=9, device="cuda")
    kc[:, :, L:L + M] = kb
    vc[:, :, L:L + M] = vb
    _, depth_m, vis = _tree_block(n_nodes, n_probes, 5, seed=77)
    depth = np.zeros((1, R), np.int32)
    depth[0, :M] = depth_m
    tree_out = _run_attention(1, q, kc, vc, _anc_words(vis)[None], depth, M, L, Hq, Hkv, h)
    rng = np.random.default_rng(0)
    for r in [0, M - 1] + [int(x) for x in rng.choice(np.arange(1, M - 1), 6, replace=False)]:
        chain = [i for i in range(M) if vis[r, i]]
        d = len(chain) - 1
        kc1, vc1 = kc.clone(), vc.clone()
        for j, i in enumerate(chain):               # ancestors become cache entries L..L+d-1, the row itself sits at L+d
            kc1[0, :, L + j] = kb[0, :, i]
            vc1[0, :, L + j] = vb[0, :, i]
        q1 = torch.zeros_like(q)
        q1[0, 0] = q[0, r]
        anc1 = np.zeros((1, R, 2), np.uint64)
        for i in range(R):
            anc1[0, i, i // 64] = np.uint64(1) << np.uint64(i % 64)
        alone = _run_attention(1, q1, kc1, vc1, anc1, np.zeros((1, R), np.int32), 1, L + d, Hq, Hkv, h)
        assert torch.equal(alone[0, 0], tree_out[0, r]), f"row {r} (depth {d})"


def test_tree_attention_one_item_and_persistent_kernels_agree_bitwise():
    """The cache below T0 is summed by one of two tensor-core kernels, picked by the number of (split, KV head,
    row tile, sequence) items in the launch.  The split length is a function of capacity, batch and head count, so
    the two are compared inside one batch: 12 sequences at KV 2048 get one split each; with 68 rows (3 row tiles)
    that is 288 items, above the switch, with the block cut to its first 20 rows (1 row tile, ancestors are
    earlier rows) 96 items, below it.  The 20 rows must come out bit for bit alike from both calls, every copy of
    a sequence like the others, and a different sequence in the same call must not disturb them."""
    Hq, Hkv, h, n_nodes, n_probes, L, few = 32, 8, 128, 64, 4, 2048, 20
    M = n_nodes + n_probes
    cap = L + R
    q, kc, vc, kb, vb = synth.random_qkv((1, R, Hq, h), (1, Hkv, cap, h), (1, Hkv, M, h), seed=77, device="cuda")
    kc[:, :, L:L + M] = kb
    vc[:, :, L:L + M] = vb
    _, d, vis = _tree_block(n_nodes, n_probes, 5, seed=5)
    assert not vis[:few, few:].any()
    anc = _anc_words(vis)[None]
    depth = np.zeros((1, R), np.int32)
    depth[0, :M] = d
    q2, kc2, vc2, _, _ = synth.random_qkv((1, R, Hq, h), (1, Hkv, cap, h), (1, Hkv, M, h), seed=78, device="cuda")
    order = [0, 1] + [0] * 10
    qq = torch.cat([(q, q2)[i] for i in order]).contiguous()
    kk = torch.cat([(kc, kc2)[i] for i in order]).contiguous()
    vv = torch.cat([(vc, vc2)[i] for i in order]).contiguous()
    ancs, depths = np.repeat(anc, len(order), 0), np.repeat(depth, len(order), 0)
    many = _run_attention(1, qq, kk, vv, ancs, depths, M, L, Hq, Hkv, h)
    anc_few = ancs.copy()
    for r in range(few, M):
        anc_few[:, r] = 0
        anc_few[:, r, r // 64] = np.uint64(1) << np.uint64(r % 64)
    fewer = _run_attention(1, qq, kk, vv, anc_few, depths, few, L, Hq, Hkv, h)
    for s in range(len(order)):
        assert torch.equal(many[s, :few], fewer[s, :few]), f"sequence {s}: the two kernels differ"
        if s >= 2:
            assert torch.equal(many[s, :M], many[0, :M]), f"copy {s}"
    assert not torch.equal(many[1, :M], many[0, :M])


def test_tree_attention_long_context_against_oracle():
    """KV length 32768 (the longest context of the batch sweep): the cache is cut in 32 splits of 1024; every
    row and head against the oracle."""
    Hq, Hkv, h, n_nodes, n_probes, L = 32, 8, 128, 64, 4, 32768
    M = n_nodes + n_probes
    cap = L + R
    q, kc, vc, kb, vb = synth.random_qkv((1, R, Hq, h), (1, Hkv, cap, h), (1, Hkv, M, h), seed=3, device="cuda")
    kc[:, :, L:L + M] = kb
    vc[:, :, L:L + M] = vb
    _, d, vis = _tree_block(n_nodes, n_probes, 5, seed=5)
    depth = np.zeros((1, R), np.int32)
    depth[0, :M] = d
    out = _run_attention(1, q, kc, vc, _anc_words(vis)[None], depth, M, L, Hq, Hkv, h)
    ref = O.tree_attention(q[0, :M].float().cpu().numpy(), kc[0, :, :L].float().permute(1, 0, 2).cpu().numpy(),
                           vc[0, :, :L].float().permute(1, 0, 2).cpu().numpy(), kb[0].float().permute(1, 0, 2).cpu().numpy(),
                           vb[0].float().permute(1, 0, 2).cpu().numpy(), vis)
    got = out[0, :M].float().cpu().numpy()
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= 2e-2


def test_bounded_wait_gives_up_and_leaves_the_context_usable():
    """A barrier that nothing signals: the kernel's wait must run out (about 50 ms), report the wait-timeout
    code through the error word and return; the next kernel on the same context works."""
    import time
    scratch = torch.zeros(256, dtype=torch.uint8, device="cuda")
    t0 = time.perf_counter()
    status = P.esp_debug_wait_selftest(scratch)
    dt = time.perf_counter() - t0
    assert status == 1                      # DEV_E_WAIT_TIMEOUT
    assert 0.03 < dt < 2.0
    g = torch.Generator().manual_seed(1)
    x = torch.randn(4, 64, generator=g).bfloat16()
    w = (torch.randn(128, 64, generator=g) * 0.05).bfloat16().cuda()
    got = _gemm(0, x, w, 4)
    ref = O.linear(x.float().numpy(), w.cpu())
    assert np.abs(got - ref).max() <= 2e-5 * np.abs(ref).max()
