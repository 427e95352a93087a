"""Host-side bookkeeping of the library, exercised without a GPU through ONELA_FLAG_DRY_RUN
(validate and advance the state machine, launch nothing): call order, slot numbering, capacity
limits, workspace carve-up and the resident-byte statistics."""
import json
from pathlib import Path

import numpy as np
import pytest

import paper_2609_12399_b200 as P
from paper_2609_12399_b200 import accounting, binding, build

GOLDEN = Path(__file__).parent / "golden"
FAKE = 4096  # a non-null, 16-byte aligned fake device address; dry runs never dereference it


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def ctx(R=2, L=2, H=4, dk=32, dv=32, W=8, steps=3, slots=64, rec="fp32", out="fp32"):
    cfg = P.make_config(R, L, H, dk, dv, W, steps, rec, out, slots, P.FLAG_DRY_RUN)
    return P.Onela(cfg, device="cpu")


def raises(status):
    class _Ctx:
        def __enter__(self):
            return self
        def __exit__(self, et, ev, tb):
            assert et is binding.OnelaError, f"expected OnelaError({status}), got {et}"
            assert ev.status == status, f"expected {status}, got {ev.status}"
            return True
    return _Ctx()


def full_step(o, req_begin, req_count, W, parents, layers):
    o.onela_reorder_beams(req_begin, req_count, parents, W)
    for l in layers:
        o.onela_append_records(req_begin, req_count, l, FAKE, FAKE, FAKE, FAKE)
        o.onela_decode_step(req_begin, req_count, l, FAKE, FAKE)


def test_invalid_configs():
    bad = [dict(num_requests=0), dict(dk=0), dict(max_beam=0), dict(arena_slots=0), dict(rec_dtype=7),
           dict(arena_slots=2 ** 31), dict(dk=36)]   # dk=36 fp32 is fine (144 B); bf16 would not be
    base = dict(num_requests=1, num_layers=1, num_heads=1, dk=32, dv=32, max_beam=4, max_steps=2, rec_dtype=0,
                out_dtype=0, arena_slots=8, flags=1)
    for i, b in enumerate(bad):
        cfg = binding.OnelaConfig(**{**base, **b})
        n = P.onela_workspace_bytes(cfg)
        if "dk" in b and b["dk"] == 36:
            assert n > 0
        else:
            assert n == 0, b
    cfg = binding.OnelaConfig(**{**base, "dk": 36, "rec_dtype": 1})   # 72-byte bf16 rows: not 16-byte vectors
    assert P.onela_workspace_bytes(cfg) == 0
    with raises(binding.E_UNSUPPORTED):                                  # sane but not compiled
        P.Onela(binding.OnelaConfig(**{**base, "dk": 48, "dv": 48}), device="cpu")
    with raises(binding.E_INVAL):                                        # misaligned workspace
        P.Onela(binding.OnelaConfig(**base), device="cpu", workspace_ptr=1024 + 16)


def test_workspace_carve_up_size():
    cfg = P.make_config(4, 16, 32, 128, 128, 512, 8, "bf16", "bf16", 4 * 512 * 8)
    n = P.onela_workspace_bytes(cfg)
    s0 = 4 * 16 * 32 * 128 * 128 * 4
    arena = 16 * 32 * (4 * 512 * 8) * 520
    tables = 4 * 2 * 8 * 512 * 4
    index = 2 * (4 * 8 * 512 * 4) + 4 * 9 * 4          # distinct-record index: positions, slot list, level offsets
    select = 4 * 256 * 1024 * 8                        # beam selection: per request 256 partial lists of 1024 candidates
    scales = 4 * 16 * 32 * 4                           # one operand scale per stored head state
    # per distinct record one beam that holds it, the per-beam positions again as bytes (rows padded), 16 bytes per record
    compact = 4 * 8 * 512 * 4 + 4 * 8 * (512 + 64) + 4 * 256 * 16
    total = s0 + arena + tables + index + select + scales + compact
    assert total <= n <= total + 13 * 1024


def test_call_order_is_enforced():
    o = ctx()
    with raises(binding.E_ORDER):
        o.onela_reorder_beams(0, 1, None, 8)                 # no shared state yet
    o.onela_init_shared_state(0, 0, FAKE)
    with raises(binding.E_ORDER):
        o.onela_append_records(0, 1, 0, FAKE, FAKE, FAKE, FAKE)   # no decode call opened
    with raises(binding.E_ORDER):
        o.onela_reorder_beams(0, 1, FAKE, 8)                 # depth 0 must pass parents = NULL
    o.onela_reorder_beams(0, 1, None, 8)
    with raises(binding.E_ORDER):
        o.onela_decode_step(0, 1, 0, FAKE, FAKE)             # records not appended yet
    with raises(binding.E_ORDER):
        o.onela_append_records(0, 1, 1, FAKE, FAKE, FAKE, FAKE)   # layer 1 holds no state
    o.onela_append_records(0, 1, 0, FAKE, FAKE, FAKE, FAKE)
    with raises(binding.E_ORDER):
        o.onela_append_records(0, 1, 0, FAKE, FAKE, FAKE, FAKE)   # exactly once per call
    o.onela_decode_step(0, 1, 0, FAKE, FAKE)
    o.onela_decode_step(0, 1, 0, FAKE, FAKE)                 # any number of times
    with raises(binding.E_ORDER):
        o.onela_reorder_beams(0, 1, None, 8)                 # depth 1 needs parents
    o.onela_reorder_beams(0, 1, FAKE, 5)                     # the beam may shrink
    with raises(binding.E_ORDER):
        o.onela_reorder_beams(0, 1, FAKE, 5)                 # previous call never appended
    assert o.depth_and_width(0) == (2, 5)


def test_fused_append_decode_counts_as_the_append():
    o = ctx()
    o.onela_init_shared_state(0, 0, FAKE)
    with raises(binding.E_ORDER):
        o.onela_append_decode_step(0, 1, 0, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE)    # no decode call opened
    o.onela_reorder_beams(0, 1, None, 8)
    o.onela_append_decode_step(0, 1, 0, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE)
    with raises(binding.E_ORDER):
        o.onela_append_decode_step(0, 1, 0, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE)    # exactly one append per call
    with raises(binding.E_ORDER):
        o.onela_append_records(0, 1, 0, FAKE, FAKE, FAKE, FAKE)
    o.onela_decode_step(0, 1, 0, FAKE, FAKE)                                       # decoding again is fine
    o.onela_reorder_beams(0, 1, FAKE, 8)                                           # and the next call may open
    with raises(binding.E_INVAL):
        o.onela_append_decode_step(0, 1, 0, FAKE, FAKE, FAKE, FAKE, None, FAKE)


def test_delta_record_mode_takes_only_the_fused_call():
    """(alpha, delta, k) records (Section 3.2) are produced where the replay runs: the separate append and decode
    calls are refused, the fused call drives the same state machine; the format needs dk == dv in {32, 64, 128}."""
    cfg = P.make_config(1, 2, 4, 32, 32, 8, 3, "fp32", "fp32", 64, P.FLAG_DRY_RUN | P.FLAG_GTR_DELTA)
    o = P.Onela(cfg, device="cpu")
    assert not o.onela_uses_tensor_core_path()
    o.onela_init_shared_state(0, 0, FAKE)
    o.onela_init_shared_state(0, 1, FAKE)
    o.onela_reorder_beams(0, 1, None, 8)
    with raises(binding.E_UNSUPPORTED):
        o.onela_append_records(0, 1, 0, FAKE, FAKE, FAKE, FAKE)
    with raises(binding.E_UNSUPPORTED):
        o.onela_decode_step(0, 1, 0, FAKE, FAKE)
    o.onela_append_decode_step(0, 1, 0, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE)
    with raises(binding.E_ORDER):
        o.onela_append_decode_step(0, 1, 0, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE)    # one append per layer and call
    with raises(binding.E_ORDER):
        o.onela_reorder_beams(0, 1, FAKE, 8)                                       # layer 1 has not appended yet
    o.onela_append_decode_step(0, 1, 1, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE)
    o.onela_reorder_beams(0, 1, FAKE, 8)
    assert o.onela_get_step_base(0, 1) == 8
    for (dk, dv) in [(128, 256), (256, 256)]:
        bad = P.make_config(1, 1, 2, dk, dv, 8, 3, "bf16", "bf16", 64, P.FLAG_DRY_RUN | P.FLAG_GTR_DELTA)
        with raises(binding.E_UNSUPPORTED):
            P.Onela(bad, device="cpu")
    tc = P.make_config(1, 1, 2, 128, 128, 8, 3, "bf16", "bf16", 64, P.FLAG_DRY_RUN | P.FLAG_GTR_DELTA)
    assert P.Onela(tc, device="cpu").onela_uses_tensor_core_path()        # 128 x 128 bf16: the tcgen05 kernel replays too
    cc = P.make_config(1, 1, 2, 128, 128, 8, 3, "bf16", "bf16", 64, P.FLAG_DRY_RUN | P.FLAG_GTR_DELTA | P.FLAG_FORCE_GENERIC)
    assert not P.Onela(cc, device="cpu").onela_uses_tensor_core_path()


def test_kernel_choice_by_shape_dtype_and_flags():
    """Which decode kernel a configuration gets (onela_uses_tensor_core_path): 1 the warp-specialised tcgen05 kernel
    (dk = 128, bf16 records, any supported dv, grouped or not), 2 the tiled tcgen05 kernel (every other shape from
    64 x 64 up, either record dtype, raw or delta records), 0 CUDA cores (32 x 32, the force flag)."""
    def kernel(dk, dv, rec, flags=0, hv=0):
        cfg = P.make_config(1, 1, 2, dk, dv, 8, 3, rec, "fp32", 64, P.FLAG_DRY_RUN | flags, num_v_heads=hv)
        return P.Onela(cfg, device="cpu").onela_uses_tensor_core_path()
    for dv in (128, 256, 512):
        assert kernel(128, dv, "bf16") == 1 and kernel(128, dv, "fp32") == 2
    for dk, dv in ((64, 64), (256, 256), (256, 512)):
        assert kernel(dk, dv, "bf16") == 2 and kernel(dk, dv, "fp32") == 2
        assert kernel(dk, dv, "bf16", P.FLAG_FORCE_GENERIC) == 0
    assert kernel(32, 32, "fp32") == 0 and kernel(32, 32, "bf16") == 0
    assert kernel(128, 128, "bf16", P.FLAG_FORCE_GENERIC) == 0
    assert kernel(64, 64, "fp32", P.FLAG_GTR_DELTA) == 2 and kernel(128, 128, "bf16", P.FLAG_GTR_DELTA) == 1
    assert kernel(128, 128, "fp32", P.FLAG_GTR_DELTA) == 2 and kernel(32, 32, "fp32", P.FLAG_GTR_DELTA) == 0
    assert kernel(64, 64, "bf16", P.FLAG_GTR_DELTA | P.FLAG_FORCE_GENERIC) == 0
    assert kernel(128, 128, "bf16", hv=4) == 1 and kernel(64, 64, "bf16", hv=4) == 2 and kernel(128, 256, "fp32", hv=6) == 2


def test_select_beams_argument_checks():
    """Selection reads the request's current beam width (1, the root, before the first call), changes no state,
    and refuses widths it cannot deliver."""
    o = ctx(W=8)
    o.onela_init_shared_state(0, 0, FAKE)
    o.onela_select_beams(0, 1, FAKE, FAKE, 16, 8, FAKE, FAKE, FAKE)               # root x 16 codes -> 8 beams
    with raises(binding.E_CAPACITY):
        o.onela_select_beams(0, 1, FAKE, FAKE, 4, 8, FAKE, FAKE, FAKE)            # only 1 x 4 candidates
    with raises(binding.E_INVAL):
        o.onela_select_beams(0, 1, FAKE, FAKE, 0, 8, FAKE, FAKE, FAKE)
    with raises(binding.E_INVAL):
        o.onela_select_beams(0, 1, FAKE, None, 16, 8, FAKE, FAKE, FAKE)
    o.onela_reorder_beams(0, 1, None, 8)
    o.onela_append_records(0, 1, 0, FAKE, FAKE, FAKE, FAKE)
    o.onela_select_beams(0, 1, FAKE, FAKE, 4, 8, FAKE, FAKE, FAKE)                # now 8 x 4 candidates
    with raises(binding.E_CAPACITY):
        o.onela_select_beams(0, 1, FAKE, FAKE, 4, 33, FAKE, FAKE, FAKE)
    with raises(binding.E_CAPACITY):
        o.onela_select_beams(0, 1, FAKE, FAKE, 1024, 1025, FAKE, FAKE, FAKE)      # more survivors than the kernel keeps
    o.onela_reorder_beams(0, 1, FAKE, 8)                                          # the call order is untouched


def test_grouped_value_heads_configs():
    """num_v_heads must be a multiple of num_heads; grouped contexts take no prefill and no delta records, and count
    k once per key head in the resident bytes."""
    ok = P.make_config(1, 1, 2, 128, 128, 8, 3, "bf16", "bf16", 64, P.FLAG_DRY_RUN, num_v_heads=6)
    o = P.Onela(ok, device="cpu")
    assert o.onela_uses_tensor_core_path()                                      # 128 x 128 bf16: grouped or not
    o.onela_init_shared_state(0, 0, FAKE)
    assert o.lib.onela_prefill_shared_state(o.handle, 0, 0, FAKE, FAKE, FAKE, FAKE, 4, None) == binding.E_UNSUPPORTED
    o.onela_reorder_beams(0, 1, None, 8)
    o.onela_append_decode_step(0, 1, 0, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE)
    assert o.onela_get_stats()["arena_bytes_used"] == 8 * (2 * 128 * 2 + 6 * (128 * 2 + 8))
    assert o.onela_get_stats()["s0_bytes"] == 6 * 128 * 128 * 4
    same = P.make_config(1, 1, 2, 128, 128, 8, 3, "bf16", "bf16", 64, P.FLAG_DRY_RUN, num_v_heads=2)
    assert P.Onela(same, device="cpu").onela_uses_tensor_core_path()           # 2 value heads on 2 key heads: not grouped
    assert P.onela_workspace_bytes(P.make_config(1, 1, 2, 128, 128, 8, 3, "bf16", "bf16", 64, 0, num_v_heads=3)) == 0
    for kw in (dict(flags=P.FLAG_DRY_RUN | P.FLAG_GTR_DELTA), dict(dk=32, dv=32)):
        args = dict(dk=128, dv=128, flags=P.FLAG_DRY_RUN)
        args.update(kw)
        bad = P.make_config(1, 1, 2, args["dk"], args["dv"], 8, 3, "fp32", "fp32", 64, args["flags"], num_v_heads=4)
        with raises(binding.E_UNSUPPORTED):
            P.Onela(bad, device="cpu")


def test_every_layer_with_state_must_append_before_next_call():
    o = ctx()
    o.onela_init_shared_state(0, 0, FAKE)
    o.onela_init_shared_state(0, 1, FAKE)
    o.onela_reorder_beams(0, 1, None, 4)
    o.onela_append_records(0, 1, 0, FAKE, FAKE, FAKE, FAKE)
    with raises(binding.E_ORDER):
        o.onela_reorder_beams(0, 1, FAKE, 4)                 # layer 1 would have a hole in its chains
    o.onela_append_records(0, 1, 1, FAKE, FAKE, FAKE, FAKE)
    o.onela_reorder_beams(0, 1, FAKE, 4)


def test_slot_numbering_bump_cursor():
    o = ctx(R=3, slots=200)
    for r in range(3):
        o.onela_init_shared_state(r, 0, FAKE)
    full_step(o, 0, 2, 8, None, [0])          # requests 0,1 batched: bases 0, 8
    full_step(o, 2, 1, 6, None, [0])          # request 2 alone: base 16
    full_step(o, 0, 2, 4, FAKE, [0])          # bases 22, 26
    full_step(o, 2, 1, 6, FAKE, [0])          # base 30
    assert [o.onela_get_step_base(0, t) for t in (0, 1)] == [0, 22]
    assert [o.onela_get_step_base(1, t) for t in (0, 1)] == [8, 26]
    assert [o.onela_get_step_base(2, t) for t in (0, 1)] == [16, 30]
    with raises(binding.E_INVAL):
        o.onela_get_step_base(0, 2)
    st = o.onela_get_stats()
    assert st["arena_bytes_used"] == 36 * 4 * 264 * 2         # slots * heads * record bytes * layers
    assert st["index_bytes"] == (4 * 2 + 4 * 2 + 6 * 2) * 4
    assert st["s0_bytes"] == 3 * 4 * 32 * 32 * 4


def test_batches_must_be_uniform_and_bounded():
    o = ctx(R=3, slots=200)
    for r in range(3):
        o.onela_init_shared_state(r, 0, FAKE)
    full_step(o, 0, 1, 8, None, [0])
    with raises(binding.E_INVAL):
        o.onela_reorder_beams(0, 2, FAKE, 8)      # request 1 is at depth 0, request 0 at depth 1
    with raises(binding.E_INVAL):
        o.onela_reorder_beams(2, 2, None, 8)      # runs past the last request
    with raises(binding.E_INVAL):
        o.onela_reorder_beams(0, 0, None, 8)
    with raises(binding.E_INVAL):
        o.onela_decode_step(0, 1, 5, FAKE, FAKE)  # no such layer
    with raises(binding.E_INVAL):
        o.onela_decode_step(0, 1, 0, FAKE + 4, FAKE)   # misaligned pointer
    with raises(binding.E_INVAL):
        o.onela_decode_step(0, 1, 0, None, FAKE)


def test_capacity_limits():
    o = ctx(R=1, W=8, steps=2, slots=12)
    o.onela_init_shared_state(0, 0, FAKE)
    with raises(binding.E_CAPACITY):
        o.onela_reorder_beams(0, 1, None, 9)      # wider than max_beam
    full_step(o, 0, 1, 8, None, [0])
    with raises(binding.E_CAPACITY):
        o.onela_reorder_beams(0, 1, FAKE, 8)      # 8 + 8 > 12 arena slots
    full_step(o, 0, 1, 4, FAKE, [0])
    with raises(binding.E_CAPACITY):
        o.onela_reorder_beams(0, 1, FAKE, 1)      # max_steps reached (checked before the arena)
    o.onela_reset()
    assert o.onela_get_stats() == {"s0_bytes": 0, "arena_bytes_used": 0, "index_bytes": 0}
    with raises(binding.E_ORDER):
        o.onela_reorder_beams(0, 1, None, 8)      # reset forgot the shared state too
    o.onela_init_shared_state(0, 0, FAKE)
    full_step(o, 0, 1, 8, None, [0])
    assert o.onela_get_step_base(0, 0) == 0       # the cursor was rewound


def test_new_prompt_restarts_a_request():
    o = ctx(R=1, slots=100)
    o.onela_init_shared_state(0, 0, FAKE)
    o.onela_init_shared_state(0, 1, FAKE)
    full_step(o, 0, 1, 8, None, [0, 1])
    full_step(o, 0, 1, 8, FAKE, [0, 1])
    o.onela_init_shared_state(0, 0, FAKE)         # a new prompt arrives in this slot
    assert o.depth_and_width(0) == (0, 0)
    o.onela_reorder_beams(0, 1, None, 8)          # depth 0 again: parents = NULL
    with raises(binding.E_ORDER):
        o.onela_append_records(0, 1, 1, FAKE, FAKE, FAKE, FAKE)   # layer 1's old state was dropped
    assert o.onela_get_step_base(0, 0) == 16      # the arena is append-only: no slot is reused


def test_batched_state_store_covers_every_layer_of_the_range():
    """onela_init_shared_states stores all layers of a range of requests: afterwards each of them may decode on
    every layer, a request outside the range may not, and a request that had decoded restarts at depth 0."""
    o = ctx(R=3, L=2, slots=100)
    for bad in [(-1, 1), (0, 0), (2, 2), (3, 1)]:
        with raises(binding.E_INVAL):
            o.onela_init_shared_states(bad[0], bad[1], FAKE)
    with raises(binding.E_INVAL):
        o.onela_init_shared_states(0, 2, 0)            # null pointer
    with raises(binding.E_INVAL):
        o.onela_init_shared_states(0, 2, FAKE + 4)     # not 16-byte aligned
    o.onela_init_shared_states(1, 2, FAKE)
    full_step(o, 1, 2, 8, None, [0, 1])
    with raises(binding.E_ORDER):
        o.onela_reorder_beams(0, 1, None, 8)            # request 0 has no state
    assert o.depth_and_width(1) == (1, 8) and o.depth_and_width(2) == (1, 8)
    o.onela_init_shared_states(2, 1, FAKE)              # a new prompt in slot 2 only
    assert o.depth_and_width(2) == (0, 0) and o.depth_and_width(1) == (1, 8)
    full_step(o, 2, 1, 8, None, [0, 1])


def test_released_slots_are_reused_lowest_first():
    o = ctx(R=3, L=1, slots=64, W=8)
    for r in range(3):
        o.onela_init_shared_state(r, 0, FAKE)
    for r in range(3):                                   # bases 0, 8, 16 and then 24, 32, 40
        full_step(o, r, 1, 8, None, [0])
    for r in range(3):
        full_step(o, r, 1, 8, FAKE, [0])
    assert [o.onela_get_step_base(r, t) for r in range(3) for t in range(2)] == [0, 24, 8, 32, 16, 40]
    used = lambda: o.onela_get_stats()["arena_bytes_used"] // (4 * (64 * 4 + 8))   # slots, from the resident bytes
    assert used() == 48
    o.onela_release_request(1)                           # frees [8, 16) and [32, 40)
    assert used() == 32 and o.depth_and_width(1) == (0, 0)
    with raises(binding.E_ORDER):
        o.onela_reorder_beams(1, 1, None, 8)             # its states went with it
    o.onela_init_shared_state(1, 0, FAKE)
    o.onela_reorder_beams(1, 1, None, 4)                 # 4 slots: the lowest hole, [8, 12)
    assert o.onela_get_step_base(1, 0) == 8
    o.onela_append_records(1, 1, 0, FAKE, FAKE, FAKE, FAKE)
    o.onela_reorder_beams(1, 1, FAKE, 8)                 # 8 slots do not fit [12, 16): the next hole, [32, 40)
    assert o.onela_get_step_base(1, 1) == 32
    o.onela_append_records(1, 1, 0, FAKE, FAKE, FAKE, FAKE)
    o.onela_reorder_beams(1, 1, FAKE, 8)                 # no hole left that fits: the cursor, [48, 56)
    assert o.onela_get_step_base(1, 2) == 48
    o.onela_release_request(2)                           # [16, 24) merges with [12, 16); [40, 48) stays apart
    o.onela_release_request(1)                           # [8, 12) merges in front; [32, 40) + [40, 48) + [48, 56) reach the
    o.onela_release_request(0)                           # cursor and lower it; request 0 then empties the arena
    assert used() == 0
    o.onela_init_shared_state(0, 0, FAKE)
    o.onela_reorder_beams(0, 1, None, 8)
    assert o.onela_get_step_base(0, 0) == 0              # back to a clean bump allocator


def test_batched_reorder_that_does_not_fit_changes_nothing():
    o = ctx(R=2, L=1, slots=20, W=8)
    for r in range(2):
        o.onela_init_shared_state(r, 0, FAKE)
    full_step(o, 0, 2, 8, None, [0])                     # 16 of 20 slots
    with raises(binding.E_CAPACITY):
        o.onela_reorder_beams(0, 2, FAKE, 8)             # the first request would fit nowhere either: nothing moves
    assert o.depth_and_width(0) == (1, 8) and o.depth_and_width(1) == (1, 8)
    o.onela_reorder_beams(0, 2, FAKE, 2)                 # 4 more slots do
    assert [o.onela_get_step_base(r, 1) for r in range(2)] == [16, 18]


def test_storage_arithmetic_matches_section_4_4():
    """The resident-byte arithmetic reproduces the capacities and write volumes the paper prints, with
    the paper's 516-byte record; the raw (k, v, alpha, beta) record kept here is 520 bytes."""
    g = json.loads((GOLDEN / "storage_section44.json").read_text())
    geo = g["geometry"]
    MiB = 2.0 ** 20
    for case in g["cases"]:
        p = accounting.persistent_bytes(T=case["T"], rec_bytes=g["paper_record_bytes"], **geo)
        # printed to three significant figures (36.25 -> 36.3, 100.75 -> 101, 32.25 -> 32.3, 96.75 -> 96.8)
        assert p["total"] / MiB == pytest.approx(case["capacity_MiB"], abs=0.0501 if case["capacity_MiB"] < 100 else 0.501)
        assert p["writes"] / MiB == pytest.approx(case["writes_MiB"], abs=0.0501)
        assert p["fullstate"] / p["total"] == pytest.approx(case["capacity_reduction"], rel=5e-3)
        assert p["fullstate_writes"] / p["writes"] == pytest.approx(case["write_reduction"], rel=5e-3)
        # the library's own statistics for the same geometry with its 520-byte records
        o = ctx(R=geo["R"], L=1, H=geo["H"], dk=128, dv=128, W=geo["W"], steps=case["T"],
                slots=geo["R"] * geo["W"] * case["T"], rec="bf16", out="bf16")
        for r in range(geo["R"]):
            o.onela_init_shared_state(r, 0, FAKE)
        for t in range(case["T"]):
            full_step(o, 0, geo["R"], geo["W"], None if t == 0 else FAKE, [0])
        st = o.onela_get_stats()
        assert st["s0_bytes"] == 4 * 2 ** 20
        assert st["arena_bytes_used"] == int(case["T"] * 16.25 * 2 ** 20)
        mine = accounting.persistent_bytes(T=case["T"], rec_bytes=accounting.record_bytes(128, 128, 2), **geo)
        assert st["s0_bytes"] + st["arena_bytes_used"] == mine["total"]
        assert st["index_bytes"] == geo["R"] * geo["W"] * case["T"] * 4


def test_distinct_record_count():
    parents = [None, np.array([0, 0, 2, 2]), np.array([1, 1, 1, 3])]
    assert accounting.distinct_records(parents, [4, 4, 4]) == [2, 2, 4]
    rows = accounting.chain_table(parents, [4, 4, 4])
    assert rows.tolist() == [[0, 1, 0], [0, 1, 1], [0, 1, 2], [2, 3, 3]]
    b = accounting.decode_bytes(R=1, H=2, dk=128, dv=128, W=4, depth=3, elem_bytes=2, out_bytes=2,
                                distinct_per_request=[8])
    assert b["algorithmic"] == 2 * 128 * 128 * 4 + 4 * 2 * 512 + 4 * 3 * 4 + 8 * 2 * 520
    assert b["undeduplicated"] == 2 * 128 * 128 * 4 + 4 * 2 * 512 + 4 * 3 * 4 + 12 * 2 * 520
