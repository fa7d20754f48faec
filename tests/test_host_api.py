"""Host-side logic of the C-ABI library, no GPU needed: the library loads and
exports every symbol the header declares, routing maps, byte accounting,
argument errors, the split-K work partition."""
import ctypes
import itertools
import math
import os
import random

import pytest

import paper_2604_22782_b200 as skv
from paper_2604_22782_b200 import binding as B


def test_library_loads_and_exports_every_declared_symbol():
    names = skv.exported_symbols()
    assert len(names) >= 20 and "skv_decode_attn" in names and "skv_append" in names and "skv_cache_create" in names
    raw = ctypes.CDLL(skv.lib_path())
    for n in names:
        assert hasattr(raw, n), n


def test_strerror_covers_all_codes():
    seen = {skv.skv_strerror(c) for c in range(0, -10, -1)}
    assert len(seen) == 10 and "unknown status" not in seen
    assert skv.skv_strerror(-99) == "unknown status"


def test_routing_from_owners_is_eq_3_2():
    """Figure 4 and an exhaustive check against a set-based restatement of Eq. (3.2)."""
    assert skv.skv_routing_from_owners(5, [0, 2]) == [0, 0, 2, 2, 2]
    L = 6
    for k in range(1, L + 1):
        for S in itertools.combinations(range(L), k):
            if 0 not in S:
                with pytest.raises(skv.SkvError) as e:
                    skv.skv_routing_from_owners(L, list(S))
                assert e.value.status == B.SKV_ERR_ROUTING
                continue
            want = [l if l in S else max(j for j in S if j < l) for l in range(L)]
            assert skv.skv_routing_from_owners(L, list(reversed(S))) == want


def test_routing_groups():
    assert skv.skv_routing_groups(8, 4) == [0, 0, 0, 0, 4, 4, 4, 4]
    assert skv.skv_routing_groups(36, 8)[-4:] == [32, 32, 32, 32]
    assert skv.skv_routing_groups(5, 1) == [0, 1, 2, 3, 4]
    with pytest.raises(skv.SkvError):
        skv.skv_routing_groups(5, 0)


def test_library_and_oracle_agree_on_routing_maps():
    from oracle import group_map, mu_from_owners
    for L, g in ((32, 2), (36, 4), (36, 8), (32, 1), (7, 3)):
        assert skv.skv_routing_groups(L, g) == group_map(L, g)
    rnd = random.Random(3)
    for _ in range(50):
        L = rnd.randint(1, 40)
        S = sorted({0} | {rnd.randrange(L) for _ in range(rnd.randint(0, L))})
        assert skv.skv_routing_from_owners(L, S) == mu_from_owners(L, S)


@pytest.mark.parametrize("r,err", [
    ([1, 1], B.SKV_ERR_ROUTING),            # layer 0 must own
    ([0, 2, 2], B.SKV_ERR_ROUTING),         # r[l] > l
    ([0, -1], B.SKV_ERR_ROUTING),
    ([0, 0, 1], B.SKV_ERR_ROUTING),         # reads a layer that keeps no cache
])
def test_bad_routing_maps_are_rejected(r, err):
    with pytest.raises(skv.SkvError) as e:
        skv.SkvCache(r, 8, 128, 16, 10, accounting_only=True)
    assert e.value.status == err


def test_unsupported_shapes_are_rejected():
    for kw in (dict(head_dim=96), dict(page_size=32), dict(head_dim=256)):
        args = dict(kv_heads=8, head_dim=128, page_size=16, max_pages=10)
        args.update(kw)
        with pytest.raises(skv.SkvError) as e:
            skv.SkvCache([0, 0], accounting_only=True, **args)
        assert e.value.status == B.SKV_ERR_UNSUPPORTED
    with pytest.raises(skv.SkvError) as e:
        skv.SkvCache([0, 0], 8, 128, 16, 0, accounting_only=True)
    assert e.value.status == B.SKV_ERR_ARG


def test_bytes_per_token_printed_values():
    """512 KB (Llama-2-7B), 128 KB (Llama-3-8B), 144 KB (Qwen3-8B) per token at full retention (Section 1)."""
    for L, Hkv, D, kb in ((32, 32, 128, 512), (32, 8, 128, 128), (36, 8, 128, 144)):
        c = skv.SkvCache(list(range(L)), Hkv, D, 16, 1, accounting_only=True)
        assert c.skv_cache_stats()["bytes_per_token"] == kb * 1024


def test_cache_bytes_scale_exactly_with_owner_fraction():
    """Owner fractions 100/50/25/12.5 % on the Llama-3-8B shape: bytes in ratio 32:16:8:4 (Section 4.3, 1/g)."""
    max_pages = 12345
    got = []
    for g in (1, 2, 4, 8):
        r = skv.skv_routing_groups(32, g)
        c = skv.SkvCache(r, 8, 128, 16, max_pages, accounting_only=True)
        st = c.skv_cache_stats()
        assert st["n_owners"] == 32 // g
        assert st["page_bytes"] == 2 * 16 * 8 * 128 * 2
        assert st["kv_bytes"] == st["n_owners"] * max_pages * st["page_bytes"]
        assert skv.skv_cache_pool_bytes(r, 8, 128, 16, max_pages) == st["kv_bytes"] + 256
        assert st["bytes_per_token"] * 16 == st["page_bytes"] * st["n_owners"]
        got.append(st["kv_bytes"])
    assert [got[0] // x for x in got] == [1, 2, 4, 8] and all(got[0] % x == 0 for x in got)


def test_library_and_oracle_agree_on_cache_bytes():
    from oracle import cache_bytes
    for g in (1, 2, 4, 8):
        r = skv.skv_routing_groups(36, g)
        pages = 517
        c = skv.SkvCache(r, 8, 128, 16, pages, accounting_only=True)
        assert c.skv_cache_stats()["kv_bytes"] == cache_bytes(r, 8, 128, 2, pages * 16)


def test_tables_4_and_5_kv_cache_cells_from_the_library():
    """KV-cache MB of Tables 4/5 (Section 4.3) from the allocator's own accounting:
    bytes_per_token * tokens, MB = 2^20, tokens = batch * (input + generated)."""
    gold = os.path.join(os.path.dirname(__file__), "golden", "table4_table5_kv_mb.txt")
    gen = {"4": 128, "5": 63}
    for ln in open(gold):
        if ln.startswith("#") or not ln.strip():
            continue
        tab, T, batch, g, mb = ln.split()
        c = skv.SkvCache(skv.skv_routing_groups(36, int(g)), 8, 128, 16, 1, accounting_only=True)
        nbytes = c.skv_cache_stats()["bytes_per_token"] * int(batch) * (int(T) + gen[tab])
        assert math.floor(nbytes / 2 ** 20 + 0.5) == int(mb)


def test_accounting_only_handle_refuses_to_launch():
    c = skv.SkvCache([0, 0], 2, 64, 16, 4, accounting_only=True)
    assert c.skv_is_owner(0) and not c.skv_is_owner(1) and c.skv_layer_owner(1) == 0
    with pytest.raises(skv.SkvError) as e:
        c.skv_layer_owner(2)
    assert e.value.status == B.SKV_ERR_LAYER
    # non-owner append is a no-op even here; an owner append needs device memory
    c.skv_append(1, None, None, None, n_tokens=3)
    with pytest.raises(skv.SkvError) as e:
        c.skv_append(0, None, None, None, n_tokens=3)
    assert e.value.status == B.SKV_ERR_ARG
    with pytest.raises(skv.SkvError) as e:
        c.skv_append(5, None, None, None, n_tokens=3)
    assert e.value.status == B.SKV_ERR_LAYER
    assert c.skv_launch_count() == 0
    assert c.skv_decode_workspace_bytes(4, 4) > 0
    with pytest.raises(skv.SkvError) as e:
        c.skv_decode_workspace_bytes(4, 3)          # 3 query heads over 2 kv heads
    assert e.value.status == B.SKV_ERR_UNSUPPORTED


def test_settings_reject_values_outside_their_range():
    """The launch-shape and merge settings take effect on the host only: bad values are SKV_ERR_ARG."""
    c = skv.SkvCache([0, 0], 2, 64, 16, 4, accounting_only=True)
    for mode in (0, 1, 2):
        c.skv_set_decode_merge(mode)
    for bad in (-1, 3):
        with pytest.raises(skv.SkvError) as e:
            c.skv_set_decode_merge(bad)
        assert e.value.status == B.SKV_ERR_ARG
    c.skv_set_decode_worker(2, 8, 16, 1)
    for bad in ((4, 8, 16, 1), (2, 9, 16, 1), (2, 8, 1, 1), (2, 8, 27, 1), (2, 8, 16, 5)):
        with pytest.raises(skv.SkvError) as e:
            c.skv_set_decode_worker(*bad)
        assert e.value.status == B.SKV_ERR_ARG
    for bad in (-1, 2):
        with pytest.raises(skv.SkvError) as e:
            c.skv_set_decode_early_fetch(bad)
        assert e.value.status == B.SKV_ERR_ARG
    # the workspace holds one 8-byte tag per partial slot next to the partials themselves
    small, large = c.skv_decode_workspace_bytes(4, 4), c.skv_decode_workspace_bytes(8, 4)
    assert large > small > 0


def test_work_partition_is_a_balanced_exact_cover():
    rnd = random.Random(1)
    cases = [(1, 1), (1, 7), (5, 7), (7, 7), (40960, 1184), (1183, 1184), (1185, 1184), (524288, 2368)]
    cases += [(rnd.randint(1, 5000), rnd.randint(1, 300)) for _ in range(30)]
    for T, Wk in cases:
        prev_end = 0
        sizes = []
        for w in range(Wk):
            b, e = B.skv_plan_worker_range(T, Wk, w)
            assert b == prev_end and e >= b
            prev_end = e
            sizes.append(e - b)
        assert prev_end == T and max(sizes) - min(sizes) <= 1
        xs = range(T) if T <= 3000 else [rnd.randrange(T) for _ in range(500)] + [0, T - 1]
        for x in xs:
            w = B.skv_plan_worker_of(T, Wk, x)
            b, e = B.skv_plan_worker_range(T, Wk, w)
            assert b <= x < e
    with pytest.raises(skv.SkvError):
        B.skv_plan_worker_of(10, 4, 10)


def test_training_time_samplers_agree_with_the_oracle():
    """R-CLA (Section 3.2) and RD-CLA@k (Section 4.2): library and oracle on the same random draws."""
    from oracle import rcla_map, rdcla_map
    rnd = random.Random(7)
    for _ in range(200):
        L = rnd.randint(1, 40)
        p = rnd.choice([0.0, 0.25, 0.5, 0.6, 0.75, 1.0])
        u = [rnd.random() for _ in range(L)]
        v = [rnd.random() for _ in range(L)]
        m = skv.skv_routing_rcla(p, u, v)
        assert m == rcla_map(p, u, v)
        assert m[0] == 0 and all(0 <= s <= l for l, s in enumerate(m))
        k = rnd.randint(1, 6)
        assert skv.skv_routing_rdcla(k, p, u) == rdcla_map(k, p, u)
    with pytest.raises(skv.SkvError):
        skv.skv_routing_rcla(0.5, [1.0], [0.0])
    with pytest.raises(skv.SkvError):
        skv.skv_routing_rcla(1.5, [0.1], [0.0])
    with pytest.raises(skv.SkvError):
        skv.skv_routing_rdcla(0, 0.5, [0.1])
