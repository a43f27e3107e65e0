"""The give-up path of the kernels' bounded waits, exercised without any fault: in the developer build of
the library (same sources, -DMASW_TRACE) one tile copy per CTA is armed on its barrier but never issued and
the wait limit is cut to a few polls, so the wait for that tile runs out.  The kernel must return, report
MASW_STATUS_WAIT_TIMEOUT in its status word, and the next normal call on the same workspace must be right."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_30252_b200 import binding, build, inputs
from helpers import assert_attention_close, dev_bf16, f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev_lib():
    build.build_trace()
    lib = binding.load_trace()
    yield lib
    binding.debug_set_wait(0, -1)


def test_product_library_has_no_developer_hooks():
    lib = binding.load()
    for name in ("masw_debug_set_trace", "masw_debug_set_wait", "masw_debug_set_flags", "masw_debug_set_verify_legacy"):
        assert not hasattr(lib, name), name


@pytest.mark.parametrize("D", [128, 64])
def test_verify_wait_runs_out_status_is_set_and_next_call_is_sound(dev_lib, D):
    """head_dim 128: the tcgen05 kernel; head_dim 64: the mma.sync kernel."""
    rng = inputs.rng_for(4, 0, 70 + D)
    B, Hq, Hkv, P, T = 1, 8, 2, 16384, 5          # 129 tiles over 64 splits: every CTA streams at least two tiles
    kb, vb = inputs.normal_bf16(rng, (B, Hkv, P + T, D)), inputs.normal_bf16(rng, (B, Hkv, P + T, D))
    qb = inputs.normal_bf16(rng, (B, T, Hq, D))
    k, v, q = dev_bf16(kb), dev_bf16(vb), dev_bf16(qb)
    kv_len = torch.tensor([P + T], dtype=torch.int32, device="cuda")
    ws = binding.verify_workspace(k, kv_len, Hq, T)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    oref, lref = oracle.verify_attend(f64(qb), f64(kb), f64(vb), [P + T])

    og, lg = binding.verify_attend(k, v, kv_len, q, workspace=ws, status=status, lib=dev_lib)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert_attention_close(og.cpu().numpy(), oref, lg.cpu().numpy(), lref, tag="developer build, normal call")

    binding.debug_set_wait(wait_limit=32, drop_tile=1)
    try:
        binding.verify_attend(k, v, kv_len, q, workspace=ws, status=status, lib=dev_lib)
        torch.cuda.synchronize()                    # the launch returns: nothing hangs, nothing traps
    finally:
        binding.debug_set_wait(0, -1)
    assert int(status.item()) & binding.STATUS_WAIT_TIMEOUT

    status.zero_()
    og, lg = binding.verify_attend(k, v, kv_len, q, workspace=ws, status=status, lib=dev_lib)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert_attention_close(og.cpu().numpy(), oref, lg.cpu().numpy(), lref, tag="call after a timed-out launch")


def test_draft_wait_runs_out_status_is_set_and_next_call_is_sound(dev_lib):
    rng = inputs.rng_for(6, 0, 75)
    L, B, Hq, Hkv, D, S, W, r = 1, 1, 8, 2, 64, 0, 8192, 8
    M = 4096
    cfg = binding.MaswConfig(L, B, Hq, Hkv, D, Hq * D, S, W, r, rollback=16, max_slots=M + 8, gamma_max=4)
    g = binding.DraftMemory(cfg, lib=dev_lib)
    o = oracle.DraftMemory(L, B, Hq, Hkv, D, S, W, r)
    t0 = S + M * r
    ks, vs = inputs.normal_bf16(rng, (B, M, Hkv, D)), inputs.normal_bf16(rng, (B, M, Hkv, D))
    kw, vw = inputs.normal_bf16(rng, (B, W, Hkv, D)), inputs.normal_bf16(rng, (B, W, Hkv, D))
    g.mem_load(0, binding.REGION_SLOT, dev_bf16(ks), dev_bf16(vs), first=0)
    g.mem_load(0, binding.REGION_LOCAL, dev_bf16(kw), dev_bf16(vw), first=t0 - W)
    g.mem_set_state(t=[t0], n_slots=[M])
    o.load_slots(0, f64(ks), f64(vs))
    zero = np.zeros((Hkv, D))
    o.raw[0][0] = [(zero, zero)] * (t0 - W) + [(f64(kw)[0, i], f64(vw)[0, i]) for i in range(W)]
    o.t, o.M = [t0], [M]
    q = inputs.normal_bf16(rng, (B, 1, Hq, D))
    k1, v1 = inputs.normal_bf16(rng, (B, 1, Hkv, D)), inputs.normal_bf16(rng, (B, 1, Hkv, D))
    o.append_raw(0, f64(k1), f64(v1))
    oref, lref = o.attend(0, f64(q))

    binding.debug_set_wait(wait_limit=32, drop_tile=1)
    try:
        g.draft_append_attend(0, dev_bf16(k1), dev_bf16(v1), dev_bf16(q))
        _, _, status = g.mem_get_state()            # synchronises: the launch returned
    finally:
        binding.debug_set_wait(0, -1)
    assert status & binding.STATUS_WAIT_TIMEOUT

    og, lg = g.draft_append_attend(0, dev_bf16(k1), dev_bf16(v1), dev_bf16(q))
    assert_attention_close(og.cpu().numpy(), oref, lg.cpu().numpy(), lref, tag="draft call after a timed-out launch")
    assert g.mem_get_state()[2] == 0               # the read above cleared the word; the sound call set nothing
    g.close()
