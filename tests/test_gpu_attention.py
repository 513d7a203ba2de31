"""GPU parity of carnator_sparse_attn against the CPU oracle, through the C ABI.

Small cases are compared element by element; the full-size workloads are run in the launch
configuration the benchmark times and compared on sampled (head, query block) rows, each of
which the oracle computes independently.
"""
import dataclasses
import os

import numpy as np
import pytest
import torch

from oracle import carnator_oracle as orc
from paper_2609_32420_b200 import carnator as cn
from paper_2609_32420_b200 import workloads as wl
from tests.gpu_util import gather_rows, o_to_host, pick_rows, to_dev
from tests.helpers import check_attention, rand_bits

pytestmark = pytest.mark.gpu

IMPLS = [cn.IMPL_PORTABLE, cn.IMPL_TCGEN05]
IMPL_IDS = ["portable", "tcgen05"]


def _tc_ok(block_q, block_k):
    return block_q == 128 and block_k == 128


def _run(Qb, Kb, Vb, N, n_text, T, Hg, Wg, bq, bk, mask, rec, impl, scale=0.0):
    B, H, _, D = Qb.shape
    Q, K, V = to_dev(Qb), to_dev(Kb), to_dev(Vb)
    shape = cn.make_shape(B, H, N, D, n_text, T, Hg, Wg, bq, bk, Q, K, V, None, softmax_scale=scale, attn_impl=impl)
    m = torch.from_numpy(mask).cuda()
    r = torch.from_numpy(rec).cuda() if rec is not None else None
    O, L, ws = cn.sparse_attn(Q, K, V, m, r, shape)
    assert cn.query_status(ws) == cn.OK, cn.last_cuda_error()
    return O, L, ws, shape


@pytest.mark.parametrize("impl", IMPLS, ids=IMPL_IDS)
def test_tiny_workload_full_compare(impl):
    w = wl.get("tiny")
    Qb, Kb, Vb = wl.gen_qkv(w)
    bp = w.build
    mask, _, _, _ = orc.build_connectivity(Qb, Kb, w.N, w.n_text, w.T, w.Hg, w.Wg, w.block, w.block, w.scale,
                                           bp.mode, bp.keep_ratio, bp.mass, bp.window_frames, bp.text_dense,
                                           bp.count_includes_forced)
    rec = wl.gen_recompute_rows(w)
    assert rec.sum() == 3
    if impl == cn.IMPL_TCGEN05:
        with pytest.raises(cn.CarnatorError) as e:
            _run(Qb, Kb, Vb, w.N, 0, w.T, w.Hg, w.Wg, 64, 64, mask, rec, impl)
        assert e.value.status == cn.ERR_UNSUPPORTED      # 64-token blocks run on the portable kernel
        return
    O, L, _, _ = _run(Qb, Kb, Vb, w.N, 0, w.T, w.Hg, w.Wg, 64, 64, mask, rec, impl)
    O_ref, L_ref = orc.attention_full(Qb, Kb, Vb, w.N, 64, 64, w.scale, mask, rec)
    check_attention(o_to_host(O), L.cpu().numpy(), O_ref, L_ref, "tiny")


CASES = [
    # name, base workload, shrink kwargs, mask density
    ("wan_ragged", "wan1p3b_480p", dict(H=2, T=3), 0.3),          # N=4680: 36 full blocks + 72-token tail, padded buffer
    ("cog_text_d64", "cogvideox5b", dict(H=3, T=2), 0.4),         # N=2926, D=64, text prefix straddles block 1
    ("hunyuan_tail16", "hunyuan_720p", dict(H=2, T=1), 0.25),     # N=3856: tail of 16 tokens
]


@pytest.mark.parametrize("impl", IMPLS, ids=IMPL_IDS)
@pytest.mark.parametrize("name,base,kw,density", CASES, ids=[c[0] for c in CASES])
def test_midsize_random_masks_full_compare(name, base, kw, density, impl):
    w = wl.shrunk(wl.get(base), **kw)
    Qb, Kb, Vb = wl.gen_qkv(w)
    mask = wl.gen_random_mask(w, density, seed=1)
    mask[0, 0, 2, :] = 0                                   # an empty row
    mask[0, 1, 3, :] = 0
    mask[0, 1, 3, w.nkb - 1] = 1                           # a row that sees only the ragged tail block
    rec = wl.gen_recompute_rows(w)
    rec[0, 2] = 0
    rec[0, 3] = 0
    O, L, ws, shape = _run(Qb, Kb, Vb, w.N, w.n_text, w.T, w.Hg, w.Wg, w.block, w.block, mask, rec, impl)
    O_ref, L_ref = orc.attention_full(Qb, Kb, Vb, w.N, w.block, w.block, w.scale, mask, rec)
    assert np.isneginf(L_ref[0, 0, 2 * w.block]).all()
    check_attention(o_to_host(O), L.cpu().numpy(), O_ref, L_ref, name)
    eff = (mask != 0) | (rec != 0)[:, None, :, None]
    assert cn.compacted_tiles(shape, ws) == int(eff.sum())


@pytest.mark.parametrize("impl", IMPLS, ids=IMPL_IDS)
@pytest.mark.parametrize("D,bq,bk,N", [(64, 64, 128, 1000), (128, 128, 64, 777), (128, 64, 64, 130),
                                       (64, 128, 128, 100), (128, 128, 128, 1), (128, 128, 128, 1153)])
def test_block_and_head_dim_combinations(D, bq, bk, N, impl):
    if impl == cn.IMPL_TCGEN05 and not _tc_ok(bq, bk):
        pytest.skip("tcgen05 kernel takes 128-token blocks")
    rng = np.random.default_rng(N + D)
    B, H = 2, 2
    Qb, Kb, Vb = (rand_bits(rng, (B, H, N, D)) for _ in range(3))
    nqb, nkb = -(-N // bq), -(-N // bk)
    mask = (rng.random((B, H, nqb, nkb)) < 0.5).astype(np.uint8)
    rec = (rng.random((B, nqb)) < 0.2).astype(np.uint8)
    O, L, _, _ = _run(Qb, Kb, Vb, N, 0, 1, 1, N, bq, bk, mask, rec, impl, scale=0.11)
    O_ref, L_ref = orc.attention_full(Qb, Kb, Vb, N, bq, bk, 0.11, mask, rec)
    check_attention(o_to_host(O), L.cpu().numpy(), O_ref, L_ref, f"D{D} bq{bq} bk{bk} N{N}")


@pytest.mark.parametrize("impl", IMPLS, ids=IMPL_IDS)
def test_degenerate_masks_and_large_scores(impl):
    rng = np.random.default_rng(5)
    N, D = 900, 128
    Qb, Kb, Vb = (rand_bits(rng, (1, 2, N, D), scale=s) for s in (4.0, 4.0, 1.0))   # scores up to ~ +-60
    nb = -(-N // 128)
    zero = np.zeros((1, 2, nb, nb), dtype=np.uint8)
    O, L, _, _ = _run(Qb, Kb, Vb, N, 0, 1, 1, N, 128, 128, zero, None, impl)
    assert (O.float() == 0).all() and torch.isneginf(L).all()           # nothing to attend to
    ones = np.ones_like(zero)
    O, L, _, _ = _run(Qb, Kb, Vb, N, 0, 1, 1, N, 128, 128, ones, None, impl)
    O_ref, L_ref = orc.attention_full(Qb, Kb, Vb, N, 128, 128, 1.0 / np.sqrt(D), ones, None)
    check_attention(o_to_host(O), L.cpu().numpy(), O_ref, L_ref, "dense, large scores")
    # recompute rows make the mask contents irrelevant
    rec = np.ones((1, nb), dtype=np.uint8)
    O2, L2, _, _ = _run(Qb, Kb, Vb, N, 0, 1, 1, N, 128, 128, zero, rec, impl)
    assert torch.equal(O, O2) and torch.equal(L, L2)


@pytest.mark.parametrize("impl", IMPLS, ids=IMPL_IDS)
def test_strided_inputs_and_rows_past_n_untouched(impl):
    """Q/K/V as slices of one packed [B, rows, 3, H, D] buffer (token-major strides); O rows >= N keep their content."""
    rng = np.random.default_rng(6)
    B, H, N, D, rows = 1, 3, 500, 128, 512
    packed = rand_bits(rng, (B, rows, 3, H, D))
    P = to_dev(packed)
    Q, K, V = (P[:, :, i].permute(0, 2, 1, 3) for i in range(3))        # [B,H,rows,D] views
    O = torch.full((B, H, rows, D), 7.0, dtype=torch.bfloat16, device="cuda")
    shape = cn.make_shape(B, H, N, D, 0, 1, 1, N, 128, 128, Q, K, V, O, attn_impl=impl)
    nb = 4
    mask = (rng.random((B, H, nb, nb)) < 0.6).astype(np.uint8)
    O, L, ws = cn.sparse_attn(Q, K, V, torch.from_numpy(mask).cuda(), None, shape, O=O)
    assert cn.query_status(ws) == cn.OK
    assert (O[:, :, N:].float() == 7.0).all()
    Qb, Kb, Vb = (np.ascontiguousarray(packed[:, :, i].transpose(0, 2, 1, 3)) for i in range(3))
    O_ref, L_ref = orc.attention_full(Qb, Kb, Vb, N, 128, 128, 1.0 / np.sqrt(D), mask, None)
    check_attention(o_to_host(O[:, :, :N]), L.cpu().numpy(), O_ref, L_ref, "strided")


def test_keys_and_values_shared_over_heads():
    """A head stride of 0 broadcasts one K / V over all heads (accepted input).  A tensor map cannot express it, so the
    call must take the portable kernel and still match the oracle; asking for the tcgen05 kernel is refused."""
    rng = np.random.default_rng(8)
    B, H, N, D = 1, 3, 700, 128
    Qb = rand_bits(rng, (B, H, N, D))
    Kb1, Vb1 = rand_bits(rng, (B, 1, N, D)), rand_bits(rng, (B, 1, N, D))
    Q, K, V = to_dev(Qb), to_dev(Kb1).expand(B, H, N, D), to_dev(Vb1).expand(B, H, N, D)
    assert K.stride(1) == 0
    nb = -(-N // 128)
    mask = (rng.random((B, H, nb, nb)) < 0.5).astype(np.uint8)
    shape = cn.make_shape(B, H, N, D, 0, 1, 1, N, 128, 128, Q, K, V, None, attn_impl=cn.IMPL_AUTO)
    O, L, ws = cn.sparse_attn(Q, K, V, torch.from_numpy(mask).cuda(), None, shape)
    assert cn.query_status(ws) == cn.OK
    O_ref, L_ref = orc.attention_full(Qb, np.repeat(Kb1, H, axis=1), np.repeat(Vb1, H, axis=1), N, 128, 128, 1.0 / np.sqrt(D), mask, None)
    check_attention(o_to_host(O), L.cpu().numpy(), O_ref, L_ref, "K/V shared over heads")
    shape.attn_impl = cn.IMPL_TCGEN05
    with pytest.raises(cn.CarnatorError) as e:
        cn.sparse_attn(Q, K, V, torch.from_numpy(mask).cuda(), None, shape)
    assert e.value.status == cn.ERR_UNSUPPORTED


# keep ratio 1.0: all-ones mask, the dense check; the HunyuanVideo-shaped layer is run at every density of its sweep
FULL = [("wan1p3b_480p", None), ("cogvideox5b", None), ("wan14b_720p", None)] + \
       [("hunyuan_720p", d) for d in wl.HUNYUAN_DENSITIES]

_full_cache = {}


def _full_inputs(name):
    """Host bits and device tensors of one full-size workload, kept while consecutive cases use the same workload."""
    if _full_cache.get("name") != name:
        _full_cache.clear()
        torch.cuda.empty_cache()
        w = wl.get(name)
        nthreads = min(16, os.cpu_count() or 1)
        host = {t: wl.gen_tensor(w, t, threads=nthreads) for t in "QKV"}
        dev = {t: to_dev(host[t]) for t in "QKV"}
        dev["Qh"], dev["Kh"] = (to_dev(wl.gen_tensor(w, t, "history", threads=nthreads)) for t in "QK")
        _full_cache.update(name=name, host=host, dev=dev)
    return _full_cache["host"], _full_cache["dev"]


@pytest.mark.parametrize("name,density", FULL, ids=[f[0] + ("" if f[1] is None else f"_{f[1]}") for f in FULL])
def test_full_size_workload_sampled_rows(name, density):
    """Whole layer at the benchmark's launch configuration (mask from the GPU builder on the historical Q/K pair).
    Every head is compared with the oracle on sampled query blocks: a recompute (forced-dense) block, the ragged
    tail block, the shortest and the longest masked row, the text blocks where there are any, and a random one."""
    w = wl.get(name)
    if density is not None:
        w = w.replace(build=dataclasses.replace(w.build, keep_ratio=density))
    host, dev = _full_inputs(name)
    Q, K, V = dev["Q"], dev["K"], dev["V"]
    shape = cn.shape_of(w, Q, K, V, None, attn_impl=cn.IMPL_AUTO)
    mask_dev, _ = cn.build_connectivity(dev["Qh"], dev["Kh"], cn.shape_of(w, dev["Qh"], dev["Kh"]), cn.params_of(w.build))
    rec = wl.gen_recompute_rows(w)
    O, L, ws = cn.sparse_attn(Q, K, V, mask_dev, torch.from_numpy(rec).cuda(), shape)
    assert cn.query_status(ws) == cn.OK, cn.last_cuda_error()
    mask = mask_dev.cpu().numpy()
    heads = [(b, h) for b in range(w.B) for h in range(w.H)]
    rows = pick_rows(mask, rec, w, heads, extra_per_head=1, seed=w.cfg)
    assert min(sum(1 for r in rows if r[:2] == bh) for bh in heads) >= 4
    O_ref, L_ref = orc.attention_rows(host["Q"], host["K"], host["V"], w.N, w.block, w.block, w.scale, mask, rec, rows)
    O_g, L_g = gather_rows(O, L, rows, w)
    check_attention(O_g, L_g, O_ref, L_ref, f"{name} keep={w.build.keep_ratio}")
    if density == 1.0:
        assert bool((mask_dev == 1).all())
    # properties that hold at any size: every valid row finite, no row past N touched is checked above by shape
    assert torch.isfinite(O.float()).all() and torch.isfinite(L).all()
    eff = (mask != 0) | (rec != 0)[:, None, :, None]
    assert cn.compacted_tiles(shape, ws) == int(eff.sum())


def test_full_size_inputs_are_released():
    _full_cache.clear()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("impl", IMPLS, ids=IMPL_IDS)
@pytest.mark.parametrize("fault", ["index", "count"])
def test_malformed_lists_are_reported_and_the_context_stays_usable(impl, fault):
    """Host-made fault: the compacted lists (or a count) are overwritten between compaction and attention.  Either
    kernel must stop the affected query block before it loads anything, report CARNATOR_ERR_DEVICE_CHECK, and leave
    the device usable."""
    rng = np.random.default_rng(21)
    B, H, N, D = 1, 1, 512, 128
    Qb, Kb, Vb = (rand_bits(rng, (B, H, N, D)) for _ in range(3))
    Q, K, V = to_dev(Qb), to_dev(Kb), to_dev(Vb)
    shape = cn.make_shape(B, H, N, D, 0, 1, 1, N, 128, 128, Q, K, V, None, attn_impl=impl)
    mask = torch.ones((B, H, 4, 4), dtype=torch.uint8, device="cuda")
    ws = cn.compact_mask(mask, None, shape)
    al = lambda x: (x + 255) // 256 * 256
    lists_off = 256 + 2 * al(4 * 4)                     # header | counts | order | lists
    lists = ws[lists_off: lists_off + 4 * 4 * 4].view(torch.int32)
    assert lists[:4].tolist() == [0, 1, 2, 3]
    if fault == "index":
        lists[1] = 1_000_000                            # row 0 now points far outside the key blocks
    else:
        counts = ws[256: 256 + 4 * 4].view(torch.int32)
        assert counts.tolist() == [4, 4, 4, 4]
        counts[2] = 9                                   # more listed blocks than there are key blocks
    O, L = cn.sparse_attn_compacted(Q, K, V, shape, ws)
    assert cn.query_status(ws) == cn.ERR_DEVICE_CHECK
    assert cn.query_status(ws) == cn.OK                 # reading the status clears it
    # the same buffers, recompacted, run normally afterwards
    ws = cn.compact_mask(mask, None, shape, ws=ws)
    O, L = cn.sparse_attn_compacted(Q, K, V, shape, ws)
    assert cn.query_status(ws) == cn.OK
    O_ref, L_ref = orc.attention_full(Qb, Kb, Vb, N, 128, 128, 1.0 / np.sqrt(D), mask.cpu().numpy(), None)
    check_attention(o_to_host(O), L.cpu().numpy(), O_ref, L_ref, "after a reported list fault")


def test_bounded_wait_runs_out_and_reports_a_timeout():
    """The wait helper of the kernels on a barrier that nothing arms, limit 1 ms: the kernel must return by itself with
    CARNATOR_ERR_DEVICE_TIMEOUT in the header, and the device must work afterwards."""
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    cn.selftest_wait_timeout(ws, 1_000_000)
    t1.record()
    assert cn.query_status(ws) == cn.ERR_DEVICE_TIMEOUT
    assert cn.query_status(ws) == cn.OK
    assert t0.elapsed_time(t1) < 500.0                 # gave up after about the limit, not after the 2 s default
    assert float(torch.ones(4, device="cuda").sum()) == 4.0


def test_withheld_tile_makes_the_attention_kernel_time_out_drain_and_return():
    """Host-made failure inside the real kernel: the header asks the K producer of the first query block to withhold its
    first copy and sets the limit of every wait to 2 ms.  The roles waiting on that tile must give up, the CTA must drain
    and free its tensor memory, the call must report CARNATOR_ERR_DEVICE_TIMEOUT, and a second, clean call on the same
    buffers must match the oracle."""
    rng = np.random.default_rng(22)
    B, H, N, D = 1, 1, 512, 128
    Qb, Kb, Vb = (rand_bits(rng, (B, H, N, D)) for _ in range(3))
    Q, K, V = to_dev(Qb), to_dev(Kb), to_dev(Vb)
    shape = cn.make_shape(B, H, N, D, 0, 1, 1, N, 128, 128, Q, K, V, None, attn_impl=cn.IMPL_TCGEN05)
    mask = torch.ones((B, H, 4, 4), dtype=torch.uint8, device="cuda")
    ws = cn.compact_mask(mask, None, shape)             # clears the header: default limit, nothing withheld
    hdr64 = ws[:256].view(torch.int64)
    hdr32 = ws[:256].view(torch.int32)
    hdr64[cn.HDR_WAIT_LIMIT_NS // 8] = 2_000_000
    hdr32[cn.HDR_DEBUG_WITHHOLD // 4] = 1
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    cn.sparse_attn_compacted(Q, K, V, shape, ws)
    t1.record()
    assert cn.query_status(ws) == cn.ERR_DEVICE_TIMEOUT
    assert "device status" in cn.last_cuda_error()
    assert t0.elapsed_time(t1) < 1000.0
    ws = cn.compact_mask(mask, None, shape, ws=ws)      # same buffers, header reset
    O, L = cn.sparse_attn_compacted(Q, K, V, shape, ws)
    assert cn.query_status(ws) == cn.OK
    O_ref, L_ref = orc.attention_full(Qb, Kb, Vb, N, 128, 128, 1.0 / np.sqrt(D), mask.cpu().numpy(), None)
    check_attention(o_to_host(O), L.cpu().numpy(), O_ref, L_ref, "after a reported time-out")


@pytest.mark.parametrize("name,kw", [("wan1p3b_480p", {}), ("tiny", {"B": 2})], ids=["wan1p3b_two_head_chunks", "tiny_two_batch_entries"])
def test_host_buffer_call_equals_device_call(name, kw):
    """carnator_sparse_attn_host works through the heads in chunks on its own copy streams; the result must be
    the device call's, bit for bit (same kernels, same inputs), with more than one chunk in flight."""
    w = wl.get(name).replace(**kw) if kw else wl.get(name)
    Qb, Kb, Vb = (wl.gen_tensor(w, t) for t in "QKV")
    if w.Nbuf != w.N:
        Qb, Kb, Vb = (np.ascontiguousarray(x[:, :, : w.N]) for x in (Qb, Kb, Vb))
    mask = wl.gen_random_mask(w, density=0.3, seed=5)
    rec = wl.gen_recompute_rows(w)
    Q, K, V = to_dev(Qb), to_dev(Kb), to_dev(Vb)
    shape = cn.shape_of(w, Q, K, V, None, attn_impl=cn.IMPL_AUTO)
    O, L, ws = cn.sparse_attn(Q, K, V, torch.from_numpy(mask).cuda(), torch.from_numpy(rec).cuda(), shape)
    assert cn.query_status(ws) == cn.OK, cn.last_cuda_error()
    pin = [torch.from_numpy(x.view(np.int16)).pin_memory() for x in (Qb, Kb, Vb)]
    hmask, hrec = torch.from_numpy(mask).pin_memory(), torch.from_numpy(rec).pin_memory()
    hO = torch.full((w.B, w.H, w.N, w.D), 0x7FC0, dtype=torch.int16).pin_memory()
    hL = torch.full((w.B, w.H, w.N), float("nan"), dtype=torch.float32).pin_memory()
    hshape = cn.shape_of(w, attn_impl=cn.IMPL_AUTO)
    arena = torch.empty(cn.attn_host_arena_bytes(hshape), dtype=torch.uint8, device="cuda")
    for _ in range(2):                       # the second call reuses the cached streams and events
        cn.sparse_attn_host(pin[0], pin[1], pin[2], hmask, hrec, hshape, hO, hL, arena)
    O_dev = O[:, :, : w.N].contiguous().view(torch.int16).cpu()
    assert torch.equal(hO, O_dev)
    assert torch.equal(hL, L[:, :, : w.N].cpu())
