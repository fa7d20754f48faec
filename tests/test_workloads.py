"""The seeded input generator: determinism, subset consistency, distribution, the
workload shapes the benchmark configurations name."""
import torch

import workloads as W


def test_values_depend_only_on_their_coordinates():
    w = W.get_workload("llama3_8b")
    si = torch.tensor([0, 3, 3, 31, 7])
    pos = torch.tensor([0, 17, 4000, 5, 123])
    K1, V1 = W.draw_kv(w, 6, si, pos)
    perm = torch.tensor([4, 2, 0, 1, 3])
    K2, V2 = W.draw_kv(w, 6, si[perm], pos[perm])
    assert torch.equal(K1[perm].view(torch.int16), K2.view(torch.int16))
    assert torch.equal(V1[perm].view(torch.int16), V2.view(torch.int16))
    K3, _ = W.draw_kv(w, 7, si, pos)
    assert not torch.equal(K1.view(torch.int16), K3.view(torch.int16))
    assert not torch.equal(K1.view(torch.int16), V1.view(torch.int16))


def test_distribution_is_standard_normal_and_q_std_is_applied():
    w = W.get_workload("qwen3_8b")
    si = torch.zeros(4096, dtype=torch.int64)
    pos = torch.arange(4096)
    K, V = W.draw_kv(w, 0, si, pos)
    for x in (K.float(), V.float()):
        assert abs(x.mean().item()) < 5e-3 and abs(x.std().item() - 1.0) < 5e-3
    Q = W.draw_q(w, 0)
    assert Q.shape == (64, 32, 128) and abs(Q.float().std().item() - 0.5) < 5e-3
    assert abs((K.float() * V.float()).mean().item()) < 5e-3


def test_workload_shapes_and_routing_maps():
    t = W.get_workload("tiny")
    assert W.routing_map(t) == [0, 0, 2, 2] and W.seq_lens(t).tolist() == [37, 128] and not t.permute_pages
    l3 = W.get_workload("llama3_8b")
    assert W.routing_map(l3) == [l - l % 2 for l in range(32)]
    n = W.seq_lens(l3)
    assert n.numel() == 32 and int(n.min()) >= 1024 and int(n.max()) <= 4096
    q = W.get_workload("qwen3_8b")
    assert sum(1 for l, r in enumerate(W.routing_map(q)) if l == r) == 9
    n = W.seq_lens(q)
    assert n.numel() == 64 and int(n.min()) >= 2048 and int(n.max()) <= 8192
    m = W.get_workload("llama2_7b_32k")
    r = W.routing_map(m)
    assert r[0] == 0 and all(r[l] <= l and r[r[l]] == r[l] for l in range(32))
    assert 8 <= sum(1 for l in range(32) if r[l] == l) <= 24
    assert W.seq_lens(m).tolist() == [32768] * 8
    for g in (1, 2, 4, 8):
        s = W.get_workload(f"sweep_g{g}")
        assert sum(1 for l, x in enumerate(W.routing_map(s)) if l == x) == 32 // g
        assert torch.equal(W.seq_lens(s), W.seq_lens(W.get_workload("sweep_g1")))


def test_page_layout_is_a_permutation_and_slots_are_unique():
    lens = torch.tensor([37, 128, 1, 0, 16], dtype=torch.int32)
    for permute in (False, True):
        table, total = W.page_layout(lens, 16, permute, seed=9)
        assert total == 3 + 8 + 1 + 0 + 1
        used = table[table >= 0]
        assert sorted(used.tolist()) == list(range(total))
        si, pos = W.token_index(lens)
        slots = W.slot_map_for(table, si, pos, 16)
        assert slots.unique().numel() == int(lens.sum())
    table, _ = W.page_layout(lens, 16, False, seed=9)
    assert table[0, :3].tolist() == [0, 1, 2] and table[1, :8].tolist() == list(range(3, 11))
