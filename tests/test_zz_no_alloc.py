"""carnator_sparse_attn_static: the form of the attention call that brings its own scratch memory.

It is meant for callers that may not allocate device memory when they call (a memory budget fixed at
start-up, a host framework that owns the allocator, a loop that cannot afford cudaMalloc's
synchronisation).  The test drives it through the C ABI and checks its output against the CPU oracle and
against the workspace form -- twice in a row with different masks, because the built-in array keeps the
previous call's lists -- that a call after the first leaves the device's free memory unchanged, and that
a shape too large for the array is refused with a clear message.

This file sorts last on purpose, so a run that stops at the first failure has already run everything else.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import carnator_oracle as orc
from paper_2609_32420_b200 import carnator as cn
from paper_2609_32420_b200 import workloads as wl
from tests.gpu_util import o_to_host, to_dev
from tests.helpers import check_attention

pytestmark = pytest.mark.gpu


def _case(w, density, seed):
    Qb, Kb, Vb = wl.gen_qkv(w)
    mask = wl.gen_random_mask(w, density, seed=seed)
    rec = wl.gen_recompute_rows(w)
    return (Qb, Kb, Vb, mask, rec), (to_dev(Qb), to_dev(Kb), to_dev(Vb), torch.from_numpy(mask).cuda(), torch.from_numpy(rec).cuda())


@pytest.mark.parametrize("name,kw", [("wan1p3b_480p", dict(H=2, T=3)), ("tiny", {})], ids=["tcgen05_path", "portable_path"])
def test_static_scratch_form_matches_workspace_form_on_two_calls_in_a_row(name, kw):
    w = wl.shrunk(wl.get(name), **kw) if kw else wl.get(name)
    for call, (density, seed) in enumerate([(0.6, 11), (0.15, 12)]):       # second call: shorter lists over stale longer ones
        (Qb, Kb, Vb, mask_np, rec_np), (Q, K, V, mask, rec) = _case(w, density, seed)
        shape = cn.shape_of(w, Q, K, V)
        O_ws, L_ws, ws = cn.sparse_attn(Q, K, V, mask, rec, shape)
        assert cn.query_status(ws) == cn.OK
        O = torch.full((w.B, w.H, w.N, w.D), float("nan"), dtype=torch.bfloat16, device="cuda")
        L = torch.full((w.B, w.H, w.N), float("nan"), dtype=torch.float32, device="cuda")
        sshape = cn.shape_of(w, Q, K, V)
        if call == 0:
            cn.sparse_attn_static(Q, K, V, mask, rec, sshape, O, L)       # first call on the device: resolves the array's address
            torch.cuda.synchronize()
        # A call after that set-up must leave the device's free memory where it was: cudaMemGetInfo sees every
        # allocation in the process, the library's own included (torch's counters would only see torch's).
        free_before, _ = torch.cuda.mem_get_info()
        cn.sparse_attn_static(Q, K, V, mask, rec, sshape, O, L)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before
        assert cn.static_status() == cn.OK
        # against the oracle, within the attention tolerances
        O_ref, L_ref = orc.attention_full(Qb, Kb, Vb, w.N, w.block, w.block, w.scale, mask_np, rec_np)
        check_attention(o_to_host(O), L.cpu().numpy(), O_ref, L_ref, f"{name} static call {call}")
        # and against the workspace form: same kernels, same lists, identical bits
        assert torch.equal(O, O_ws) and torch.equal(L, L_ws)


def test_shape_beyond_the_builtin_array_is_refused_before_any_launch():
    w = wl.get("wan14b_720p")                          # needs ~56 MB of lists; the array holds 8 MiB
    shape = cn.shape_of(w)
    assert cn.attn_workspace_bytes(shape) > cn.STATIC_SCRATCH_BYTES
    launches = cn.kernel_launches()
    dummy = torch.zeros(256, dtype=torch.uint8, device="cuda")
    p = dummy.data_ptr()
    st = cn.lib().carnator_sparse_attn_static(p, p, p, p, None, ctypes.byref(shape), p, p, None)
    assert st == cn.ERR_WORKSPACE
    assert "built-in array holds" in cn.last_cuda_error()
    assert cn.kernel_launches() == launches
