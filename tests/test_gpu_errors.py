"""Error paths of the C ABI on a GPU machine.  Every failure here is made on the host (a budget
the pool cannot cover, a host tier that is full, a closed request, a pool that is too small,
arguments that do not fit together); none of them launches a kernel with bad input.  A refused
call must leave the context as it was: the run goes on afterwards and still matches the oracle.
The one device-side case is the bounded wait: a warp polls, for a few hundred polls, a flag
that nothing raises, gives up and reports it; the context stays usable.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import workloads as W
from oracle import spin_oracle as O

pytestmark = pytest.mark.gpu


def _cfg(P, **kw):
    base = dict(device=0, num_layers=1, num_q_heads=4, num_kv_heads=2, max_requests=2, max_context_tokens=16 * 8,
                partition_kind=P.PART_PAGE_MINMAX, topk=4, lru_buckets=4, gpu_cache_pages=2 * 2 * 6, host_pages=64)
    base.update(kw)
    return P.make_config(**base)


def _kv(n, seed=0):
    g = torch.Generator(device="cpu").manual_seed(seed)
    k = torch.randn(n, 2, 128, generator=g).to(torch.bfloat16).cuda()
    v = torch.randn(n, 2, 128, generator=g).to(torch.bfloat16).cuda()
    return k, v


def test_budget_beyond_the_pool_is_refused_and_the_pool_is_untouched():
    import paper_2604_26837_b200 as P
    s = P.Spin(_cfg(P))
    r0 = s.request_open(6)
    r1 = s.request_open(6)                         # 2 requests x 2 sets x 6 pages = the whole pool
    s.request_close(r1)
    with pytest.raises(P.SpinError) as e:
        s.request_open(7)                          # 14 pages wanted, 12 free
    assert e.value.code == 5                       # SPIN_ERR_BUDGET
    assert s.stats()["gpu_pages_in_use"] == 12
    with pytest.raises(P.SpinError) as e:
        s.set_budget(r0, 13)                       # growing needs 14 more, 12 free
    assert e.value.code == 5
    assert s.request_open(6) == r1                 # the refused calls took nothing
    st = s.stats()
    assert st["gpu_pages_in_use"] == 24 and st["error_bits"] == 0 and st["kernel_launches"] == 0
    s.close()


def test_calls_on_a_closed_request_are_state_errors():
    import paper_2604_26837_b200 as P
    s = P.Spin(_cfg(P))
    r = s.request_open(4)
    k, v = _kv(20)
    s.append_kv(r, 0, k, v, 20)
    s.request_close(r)
    q = torch.zeros(1, 4, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(q)
    for call in (lambda: s.decode_step(0, [r], q, out), lambda: s.append_kv(r, 0, k, v, 20),
                 lambda: s.append_kv_batch(0, [r], k[:1], v[:1]), lambda: s.request_close(r),
                 lambda: s.set_budget(r, 2), lambda: s.decode_step_append(0, s.req_array([r]), k[:1], v[:1], q, out)):
        with pytest.raises(P.SpinError) as e:
            call()
        assert e.value.code == 2, e.value          # SPIN_ERR_STATE
    # all request slots taken
    a, b = s.request_open(1), s.request_open(1)
    with pytest.raises(P.SpinError) as e:
        s.request_open(1)
    assert e.value.code == 2
    assert s.stats()["error_bits"] == 0
    s.close()


def test_pool_too_small_and_bad_pool_pointer():
    import paper_2604_26837_b200 as P
    lib = P.load()
    cfg = _cfg(P)
    need, _ = P.spin_required_bytes(cfg)
    pool = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
    base = (pool.data_ptr() + 255) // 256 * 256
    h = C.c_void_p()
    cfg.hbm_pool, cfg.hbm_pool_bytes = base, need - 256
    assert lib.spin_create(C.byref(cfg), C.byref(h)) == 3 and not h.value       # SPIN_ERR_OOM_DEVICE
    cfg.hbm_pool, cfg.hbm_pool_bytes = base + 8, need                           # not 256-byte aligned
    assert lib.spin_create(C.byref(cfg), C.byref(h)) == 1 and not h.value
    cfg.hbm_pool, cfg.hbm_pool_bytes = None, need
    assert lib.spin_create(C.byref(cfg), C.byref(h)) == 1 and not h.value
    cfg.hbm_pool, cfg.hbm_pool_bytes = base, need
    assert lib.spin_create(C.byref(cfg), C.byref(h)) == 0 and h.value
    assert lib.spin_destroy(h) == 0


def _oracle_for(P, cfg):
    return O.SpinOracle(O.OracleConfig(cfg.num_layers, cfg.num_q_heads, cfg.num_kv_heads, 128, 16,
                                       cfg.partition_kind, cfg.topk, cfg.lru_buckets))


def test_a_full_host_tier_refuses_the_append_and_changes_nothing():
    import paper_2604_26837_b200 as P
    # 2 kv heads x 5 pages = 10 host pages: a 70-token prefill takes them all (4 full pages + tail)
    cfg = _cfg(P, host_pages=10, trace=1)
    s = P.Spin(cfg)
    orc = _oracle_for(P, cfg)
    r, ro = s.request_open(6), orc.request_open(6)
    k, v = _kv(96, seed=3)
    with pytest.raises(P.SpinError) as e:
        s.append_kv(r, 0, k, v, 96)                # 6 pages per head: more than the tier holds
    assert e.value.code == 4                       # SPIN_ERR_OOM_HOST
    assert s.stats()["host_pages_in_use"] == 0
    s.append_kv(r, 0, k[:80], v[:80], 80)          # exactly 5 pages per head
    orc.append_kv(ro, 0, W.to_bits(k[:80]), W.to_bits(v[:80]))
    assert s.stats()["host_pages_in_use"] == 10
    q = torch.randn(1, 4, 128).to(torch.bfloat16).cuda()
    out = torch.zeros_like(q)
    # the 81st token would open a sixth page: refused, by the batch form and by the fused form
    for call in (lambda: s.append_kv_batch(0, [r], k[80:81], v[80:81]),
                 lambda: s.decode_step_append(0, s.req_array([r]), k[80:81], v[80:81], q, out)):
        with pytest.raises(P.SpinError) as e:
            call()
        assert e.value.code == 4
    d = s.debug_dump(r, 0, 0, 4, 8, 6, 8)
    assert d["n_tokens"] == 80 and d["step"] == 0
    # the context still works and still agrees with the oracle
    s.decode_step(0, [r], q, out)
    ref = orc.decode_step(0, [ro], W.to_bits(q))
    torch.cuda.synchronize()
    assert np.abs(out.float().cpu().numpy() - ref).max() <= 2e-2
    for h in range(2):
        assert list(s.debug_dump(r, 0, h, 4, 8, 6, 8)["selected"]) == list(orc.last_trace[(ro, 0, h)].selected)
    st = s.stats()
    assert st["error_bits"] == 0 and st["host_pages_in_use"] == 10
    s.close()


def test_mismatched_kv_memory_kinds_are_refused_before_any_state_changes():
    import paper_2604_26837_b200 as P
    cfg = _cfg(P, host_pages=64, trace=1, max_context_tokens=16 * 12)
    s = P.Spin(cfg)
    orc = _oracle_for(P, cfg)
    reqs, oreqs = [s.request_open(5), s.request_open(5)], [orc.request_open(5), orc.request_open(5)]
    for i, (r, ro) in enumerate(zip(reqs, oreqs)):
        k, v = _kv(16 * 6 + 15, seed=10 + i)       # the next token completes a page: the append would map new entries
        s.append_kv(r, 0, k, v, k.shape[0])
        orc.append_kv(ro, 0, W.to_bits(k), W.to_bits(v))
    kn, vn = _kv(2, seed=20)
    q = torch.randn(2, 4, 128).to(torch.bfloat16).cuda()
    out = torch.zeros_like(q)
    before = s.stats()
    for call in (lambda: s.decode_step_append(0, s.req_array(reqs), kn, vn.cpu(), q, out),      # device k, host v
                 lambda: s.decode_step_append(0, s.req_array(reqs), kn.cpu(), vn, q, out),
                 lambda: s.append_kv_batch(0, reqs, kn, vn.cpu())):
        with pytest.raises(P.SpinError) as e:
            call()
        assert e.value.code == 1                   # SPIN_ERR_INVALID
    after = s.stats()
    assert after["host_pages_in_use"] == before["host_pages_in_use"] and after["kernel_launches"] == before["kernel_launches"]
    for r in reqs:
        assert s.debug_dump(r, 0, 0, 4, 8, 5, 16)["n_tokens"] == 16 * 6 + 15
    # the same step with well-formed arguments, twice (it crosses the page boundary), against the oracle
    for step in range(2):
        s.decode_step_append(0, s.req_array(reqs), kn, vn, q, out)
        for i, ro in enumerate(oreqs):
            orc.append_kv(ro, 0, W.to_bits(kn[i:i + 1]), W.to_bits(vn[i:i + 1]))
        ref = orc.decode_step(0, oreqs, W.to_bits(q))
        torch.cuda.synchronize()
        assert np.abs(out.float().cpu().numpy() - ref).max() <= 2e-2
        for i, (r, ro) in enumerate(zip(reqs, oreqs)):
            for h in range(2):
                d = s.debug_dump(r, 0, h, 4, 8, 5, 16)
                tr = orc.last_trace[(ro, 0, h)]
                assert list(d["selected"]) == list(tr.selected) and list(d["slot_partition"]) == list(tr.slot_part)
                assert d["n_tokens"] == 16 * 6 + 16 + step
    assert s.stats()["error_bits"] == 0
    s.close()


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    import paper_2604_26837_b200 as P
    cfg = _cfg(P)
    s = P.Spin(cfg)
    orc = _oracle_for(P, cfg)
    r, ro = s.request_open(4), orc.request_open(4)
    k, v = _kv(50, seed=5)
    s.append_kv(r, 0, k, v, 50)
    orc.append_kv(ro, 0, W.to_bits(k), W.to_bits(v))
    assert s.stats()["status"] == 0
    with pytest.raises(P.SpinError):
        s.debug_wait_probe(1 << 20)                # the limit itself is limited
    s.debug_wait_probe(200)                        # 200 polls of a flag that nothing raises
    st = s.stats()
    assert st["status"] == 7 and st["error_bits"] == 4 and st["first_error_site"] > 0      # SPIN_ERR_TIMEOUT / SPIN_DEV_ERR_TIMEOUT
    # the kernel returned, the context still computes the right thing (the bit is sticky)
    q = torch.randn(1, 4, 128).to(torch.bfloat16).cuda()
    out = torch.zeros_like(q)
    s.decode_step(0, [r], q, out)
    ref = orc.decode_step(0, [ro], W.to_bits(q))
    torch.cuda.synchronize()
    assert np.abs(out.float().cpu().numpy() - ref).max() <= 2e-2
    assert s.stats()["error_bits"] == 4
    s.close()
