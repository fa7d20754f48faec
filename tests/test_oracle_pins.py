"""Pins for the CPU oracle: values the paper prints, closed forms, a library
attention routine in fp64, and brute force.  None of them re-uses the oracle's
own formula; each is chosen so that a plausible mistake in the oracle (wrong
head mapping, dropped scale, wrong source layer, off-by-one length) fails."""
import itertools
import math
import os

import pytest
import torch

import workloads as W
from oracle import Oracle, cache_bytes, count_owners, group_map, mu_from_owners

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(path):
    with open(os.path.join(GOLD, path)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def _rand_bf16(shape, seed, std=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(shape, generator=g, dtype=torch.float32) * std).to(torch.bfloat16)


def _fill(o, L, B, n, Hkv, D, seed):
    """Distinct random K/V for every layer; returns dict layer -> (K,V) [B,n,Hkv,D]."""
    store = {}
    b_idx = torch.arange(B).repeat_interleave(n)
    t_idx = torch.arange(n).repeat(B)
    for l in range(L):
        K = _rand_bf16((B, n, Hkv, D), seed * 100 + 2 * l)
        V = _rand_bf16((B, n, Hkv, D), seed * 100 + 2 * l + 1)
        o.append(l, K.reshape(B * n, Hkv, D), V.reshape(B * n, Hkv, D), b_idx, t_idx)
        store[l] = (K, V)
    return store


def _sdpa64(Q, K, V, lens, scale):
    """torch's library attention in fp64, one sequence at a time.
    Q [B,Hq,D]; K,V [B,n,Hkv,D]; GQA by repeat_interleave over heads."""
    B, Hq, D = Q.shape
    Hkv = K.shape[2]
    G = Hq // Hkv
    out = torch.zeros(B, Hq, D, dtype=torch.float64)
    for b in range(B):
        n = int(lens[b])
        if n == 0:
            continue
        q = Q[b].double()[None, :, None, :]                                  # [1,Hq,1,D]
        k = K[b, :n].double().permute(1, 0, 2).repeat_interleave(G, 0)[None]  # [1,Hq,n,D]
        v = V[b, :n].double().permute(1, 0, 2).repeat_interleave(G, 0)[None]
        out[b] = torch.nn.functional.scaled_dot_product_attention(q, k, v, scale=scale)[0, :, 0, :]
    return out


# ------------------------------------------------------------------ routing
def test_fig4_sharing_example():
    """Figure 4: S={1,3} of 5 layers -> layers 1-2 read KV1, 3-5 read KV3; 60 % saved."""
    rows = {r[0]: r[1:] for r in _rows("fig4_sharing.txt")}
    L = int(rows["n_layers"][0])
    owners0 = [int(x) - 1 for x in rows["cached"]]
    reads0 = [int(x) - 1 for x in rows["reads"]]
    mu = mu_from_owners(L, owners0)
    assert mu == reads0 == [0, 0, 2, 2, 2]
    assert count_owners(mu) == 2
    full = cache_bytes(list(range(L)), 8, 128, 2, 1000)
    shared = cache_bytes(mu, 8, 128, 2, 1000)
    assert round(100 * (1 - shared / full)) == int(rows["memory_saved_percent"][0])
    num, den = rows["cached_fraction"][0].split("/")
    assert shared * int(den) == full * int(num)


def test_mu_matches_definition_on_all_small_owner_sets():
    """Eq. (3.2) by exhaustive enumeration, against an independent set-based restatement."""
    L = 6
    for k in range(1, L + 1):
        for S in itertools.combinations(range(L), k):
            got = mu_from_owners(L, S)
            if 0 not in S:
                assert got is None          # mu undefined for layers below the first owner
                continue
            want = [l if l in S else max(j for j in S if j < l) for l in range(L)]
            assert got == want
            assert all(got[got[l]] == got[l] and got[l] <= l for l in range(L))


def test_owner_reads_itself():
    """l' = l reduces to self-attention: with S = all layers mu is the identity."""
    assert mu_from_owners(7, range(7)) == list(range(7))


def test_group_maps():
    """Section 4.3 leaders: g consecutive layers share the first; 'every 4th layer' (Section 1)."""
    assert group_map(8, 4) == [0, 0, 0, 0, 4, 4, 4, 4]
    assert group_map(36, 4) == mu_from_owners(36, range(0, 36, 4))
    assert count_owners(group_map(36, 4)) == 9
    assert count_owners(group_map(36, 8)) == 5           # last group is short
    assert group_map(5, 1) == [0, 1, 2, 3, 4]


# ------------------------------------------------------------------ bytes
def test_bytes_per_token_printed_values():
    for name, L, Hkv, D, kb in _rows("kv_bytes_per_token.txt"):
        L, Hkv, D, kb = int(L), int(Hkv), int(D), int(kb)
        per_token = cache_bytes(list(range(L)), Hkv, D, 2, 1)
        assert per_token == 2 * L * Hkv * D * 2
        assert per_token // 1024 == kb and per_token % 1024 == 0


def test_tables_4_and_5_kv_cache_column():
    """KV-cache MB cells of Tables 4 and 5.  The tables do not print how many
    tokens were generated; 128 (Table 4) and 63 (Table 5) are the counts that
    reproduce every cell, with MB = 2^20 bytes and round-half-up."""
    gen = {"4": 128, "5": 63}
    for tab, T, batch, g, mb in _rows("table4_table5_kv_mb.txt"):
        r = group_map(36, int(g))
        n_tok = int(batch) * (int(T) + gen[tab])
        got = cache_bytes(r, 8, 128, 2, n_tok) / 2 ** 20
        assert math.floor(got + 0.5) == int(mb), (tab, T, batch, g, got)


def test_cache_scales_as_one_over_g():
    """'KV cache memory scales as 1/g' (Section 4.3)."""
    base = cache_bytes(group_map(32, 1), 8, 128, 2, 4096)
    for g in (2, 4, 8):
        assert cache_bytes(group_map(32, g), 8, 128, 2, 4096) * g == base


# ------------------------------------------------------------------ attention
@pytest.mark.parametrize("Hq,Hkv,D", [(4, 2, 64), (6, 2, 32), (8, 8, 16), (8, 1, 128)])
def test_identity_map_equals_library_attention(Hq, Hkv, D):
    """Identity routing = standard per-layer attention (Algorithm 1)."""
    L, B, n = 3, 3, 40
    o = Oracle(L, list(range(L)), Hq, Hkv, D, B, n)
    store = _fill(o, L, B, n, Hkv, D, seed=7)
    lens = torch.tensor([40, 1, 23], dtype=torch.int32)
    for l in range(L):
        Q = _rand_bf16((B, Hq, D), 900 + l)
        for scale in (D ** -0.5, 0.37):
            got = o.decode_attn(l, Q, lens, scale)
            want = _sdpa64(Q, store[l][0], store[l][1], lens, scale)
            assert torch.allclose(got, want, rtol=1e-12, atol=1e-13)


def test_all_layers_routed_to_layer0():
    L, B, n, Hq, Hkv, D = 4, 2, 19, 4, 2, 32
    o = Oracle(L, [0] * L, Hq, Hkv, D, B, n)
    store = _fill(o, L, B, n, Hkv, D, seed=3)
    lens = torch.tensor([19, 7], dtype=torch.int32)
    for l in range(L):
        Q = _rand_bf16((B, Hq, D), 50 + l)
        want = _sdpa64(Q, store[0][0], store[0][1], lens, D ** -0.5)
        assert torch.allclose(o.decode_attn(l, Q, lens), want, rtol=1e-12, atol=1e-13)


def test_routed_layers_read_their_source_and_nothing_else():
    """r=[0,0,2,2]: layer 1 must use layer 0's cache, layer 3 layer 2's; changing the
    non-owner layers' own K/V changes no output."""
    L, B, n, Hq, Hkv, D = 4, 2, 33, 4, 2, 64
    r = [0, 0, 2, 2]
    o = Oracle(L, r, Hq, Hkv, D, B, n)
    store = _fill(o, L, B, n, Hkv, D, seed=11)
    lens = torch.tensor([33, 20], dtype=torch.int32)
    Qs = [_rand_bf16((B, Hq, D), 70 + l) for l in range(L)]
    outs = [o.decode_attn(l, Qs[l], lens) for l in range(L)]
    for l in range(L):
        want = _sdpa64(Qs[l], store[r[l]][0], store[r[l]][1], lens, D ** -0.5)
        assert torch.allclose(outs[l], want, rtol=1e-12, atol=1e-13)
        other = _sdpa64(Qs[l], store[l][0], store[l][1], lens, D ** -0.5)
        if r[l] != l:
            assert not torch.allclose(outs[l], other, rtol=1e-3, atol=1e-3)
    # overwrite the non-owner layers' own stores: outputs must not move
    b_idx = torch.arange(B).repeat_interleave(n)
    t_idx = torch.arange(n).repeat(B)
    for l in (1, 3):
        o.append(l, _rand_bf16((B * n, Hkv, D), 999 + l), _rand_bf16((B * n, Hkv, D), 1999 + l), b_idx, t_idx)
    for l in range(L):
        assert torch.equal(o.decode_attn(l, Qs[l], lens), outs[l])


def test_single_cached_token_returns_its_value_exactly():
    L, B, Hq, Hkv, D = 2, 3, 6, 3, 16
    o = Oracle(L, [0, 0], Hq, Hkv, D, B, 4)
    store = _fill(o, L, B, 4, Hkv, D, seed=5)
    lens = torch.ones(B, dtype=torch.int32)
    out = o.decode_attn(1, _rand_bf16((B, Hq, D), 1), lens)
    V0 = store[0][1][:, 0].double()                     # [B,Hkv,D]
    assert torch.equal(out, V0.repeat_interleave(Hq // Hkv, dim=1))


def test_softmax_weights_are_a_distribution_and_uniform_for_zero_query():
    L, B, n, Hq, Hkv, D = 1, 2, 57, 4, 2, 32
    o = Oracle(L, [0], Hq, Hkv, D, B, n)
    store = _fill(o, L, B, n, Hkv, D, seed=9)
    Q = _rand_bf16((B, Hq, D), 2, std=2.0)
    for b in range(B):
        for h in range(Hq):
            w = o.attn_weights(0, Q, b, h, n)
            assert (w >= 0).all() and abs(w.sum().item() - 1.0) < 1e-15 * n
    lens = torch.tensor([57, 31], dtype=torch.int32)
    out = o.decode_attn(0, torch.zeros(B, Hq, D, dtype=torch.bfloat16), lens)
    for b in range(B):
        mean_v = store[0][1][b, : int(lens[b])].double().mean(0)          # [Hkv,D]
        assert torch.allclose(out[b], mean_v.repeat_interleave(Hq // Hkv, 0), rtol=1e-13, atol=1e-14)


def test_two_token_closed_form_sigmoid():
    """n=2 with axis-aligned vectors: w0 = 1/(1+exp(-(s0-s1))), s_t = scale*a*k_t."""
    D, scale, a, k0, k1 = 8, 0.25, 3.0, 2.0, -1.5
    o = Oracle(1, [0], 1, 1, D, 1, 2)
    K = torch.zeros(2, 1, D, dtype=torch.bfloat16)
    V = torch.zeros(2, 1, D, dtype=torch.bfloat16)
    K[0, 0, 0], K[1, 0, 0] = k0, k1
    V[0, 0, :], V[1, 0, :] = 1.0, -3.0
    o.append(0, K, V, torch.tensor([0, 0]), torch.tensor([0, 1]))
    Q = torch.zeros(1, 1, D, dtype=torch.bfloat16)
    Q[0, 0, 0] = a
    w0 = 1.0 / (1.0 + math.exp(-(scale * a * (k0 - k1))))
    out = o.decode_attn(0, Q, torch.tensor([2], dtype=torch.int32), scale)
    assert torch.allclose(out, torch.full((1, 1, D), w0 * 1.0 + (1 - w0) * -3.0, dtype=torch.float64),
                          rtol=1e-14, atol=0)


def test_brute_force_tiny():
    """Independent pure-Python loops, no max subtraction, explicit weights."""
    L, B, n, Hq, Hkv, D = 3, 2, 5, 4, 2, 4
    r = [0, 0, 2]
    o = Oracle(L, r, Hq, Hkv, D, B, n)
    store = _fill(o, L, B, n, Hkv, D, seed=21)
    lens = [5, 3]
    scale = 0.5
    for l in range(L):
        Q = _rand_bf16((B, Hq, D), 300 + l)
        got = o.decode_attn(l, Q, torch.tensor(lens, dtype=torch.int32), scale)
        Ks, Vs = store[r[l]]
        for b in range(B):
            for h in range(Hq):
                kv = h // (Hq // Hkv)
                e = []
                for t in range(lens[b]):
                    s = sum(float(Q[b, h, d]) * float(Ks[b, t, kv, d]) for d in range(D))
                    e.append(math.exp(scale * s))
                z = sum(e)
                for d in range(D):
                    want = sum(e[t] / z * float(Vs[b, t, kv, d]) for t in range(lens[b]))
                    assert abs(got[b, h, d].item() - want) < 1e-12


def test_zero_length_sequence_gives_zero_row_and_length_is_respected():
    L, B, n, Hq, Hkv, D = 1, 2, 10, 2, 1, 8
    o = Oracle(L, [0], Hq, Hkv, D, B, n)
    store = _fill(o, L, B, n, Hkv, D, seed=4)
    Q = _rand_bf16((B, Hq, D), 8)
    out = o.decode_attn(0, Q, torch.tensor([0, 6], dtype=torch.int32))
    assert torch.equal(out[0], torch.zeros(Hq, D, dtype=torch.float64))
    want = _sdpa64(Q, store[0][0], store[0][1], [0, 6], D ** -0.5)
    assert torch.allclose(out, want, rtol=1e-12, atol=1e-13)
    full = o.decode_attn(0, Q, torch.tensor([0, 7], dtype=torch.int32))
    assert not torch.allclose(full[1], out[1])


def test_append_is_a_bit_copy_and_last_write_wins():
    o = Oracle(2, [0, 0], 2, 2, 8, 2, 6)
    K = _rand_bf16((3, 2, 8), 1)
    V = _rand_bf16((3, 2, 8), 2)
    o.append(1, K, V, torch.tensor([1, 0, 1]), torch.tensor([5, 2, 5]))
    k, v = o.read(1, 1, 5)
    assert torch.equal(k.view(torch.int16), K[2].view(torch.int16))
    assert torch.equal(v.view(torch.int16), V[2].view(torch.int16))
    k, v = o.read(1, 0, 2)
    assert torch.equal(k.view(torch.int16), K[1].view(torch.int16))
    k, _ = o.read(1, 0, 0)
    assert torch.equal(k.view(torch.int16), torch.zeros(2, 8, dtype=torch.int16))
    with pytest.raises(RuntimeError):
        o.read(0, 0, 0)          # layer 0 never appended: no store


def test_oracle_on_the_tiny_workload_matches_library_attention():
    """The tiny workload end to end (shapes of the first benchmark config)."""
    w = W.get_workload("tiny")
    r = W.routing_map(w)
    lens = W.seq_lens(w)
    o = Oracle(w.n_layers, r, w.q_heads, w.kv_heads, w.head_dim, w.batch, int(lens.max()))
    si, pos = W.token_index(lens)
    dense = {}
    for l in range(w.n_layers):
        K, V = W.draw_kv(w, l, si, pos)
        o.append(l, K, V, si, pos)
        Kd = torch.zeros(w.batch, int(lens.max()), w.kv_heads, w.head_dim, dtype=torch.bfloat16)
        Vd = torch.zeros_like(Kd)
        Kd[si, pos], Vd[si, pos] = K, V
        dense[l] = (Kd, Vd)
    for l in range(w.n_layers):
        Q = W.draw_q(w, l)
        want = _sdpa64(Q, dense[r[l]][0], dense[r[l]][1], lens, w.head_dim ** -0.5)
        assert torch.allclose(o.decode_attn(l, Q, lens), want, rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ do the pins bite?
class _Mutant(Oracle):
    """The oracle with one plausible mistake planted on the CPU side of its interface."""

    def __init__(self, mistake, *a, **k):
        super().__init__(*a, **k)
        self.mistake = mistake

    def append(self, layer, K, V, seq_idx, pos):
        if self.mistake == "swap_kv":
            K, V = V, K
        super().append(layer, K, V, seq_idx, pos)

    def decode_attn(self, layer, Q, seq_lens, scale=None):
        scale = self.D ** -0.5 if scale is None else scale
        if self.mistake == "no_scale":
            scale = 1.0
        if self.mistake == "short_by_one":
            seq_lens = (seq_lens - 1).clamp(min=0)
        if self.mistake == "own_layer":          # ignores the routing map: reads the layer's own store
            return self._identity_twin.decode_attn(layer, Q, seq_lens, scale)
        if self.mistake == "head_mod":           # query head h reads kv head h % Hkv instead of h // G
            G = self.Hq // self.Hkv
            perm = torch.tensor([(h % self.Hkv) * G + h // self.Hkv for h in range(self.Hq)])
            inv = torch.empty_like(perm)
            inv[perm] = torch.arange(self.Hq)
            return super().decode_attn(layer, Q[:, inv].contiguous(), seq_lens, scale)[:, perm]
        return super().decode_attn(layer, Q, seq_lens, scale)


def _pins_hold(make):
    """A small set of the pins above, as one predicate over an oracle constructor."""
    L, B, n, Hq, Hkv, D = 4, 2, 12, 4, 2, 16
    r = [0, 0, 2, 2]
    o = make(L, r, Hq, Hkv, D, B, n)
    twin = Oracle(L, list(range(L)), Hq, Hkv, D, B, n)
    store = _fill(o, L, B, n, Hkv, D, seed=11)
    _fill(twin, L, B, n, Hkv, D, seed=11)
    o._identity_twin = twin
    lens = torch.tensor([12, 5], dtype=torch.int32)
    ok = True
    for l in range(L):
        Q = _rand_bf16((B, Hq, D), 70 + l)
        want = _sdpa64(Q, store[r[l]][0], store[r[l]][1], lens, D ** -0.5)     # library attention on the source layer
        ok &= torch.allclose(o.decode_attn(l, Q, lens), want, rtol=1e-12, atol=1e-13)
    one = torch.tensor([1, 1], dtype=torch.int32)                               # a single cached token returns its V
    got = o.decode_attn(0, _rand_bf16((B, Hq, D), 5), one)
    ok &= torch.equal(got, store[0][1][:, 0].double().repeat_interleave(Hq // Hkv, 1))
    return bool(ok)


def test_planted_mistakes_fail_the_pins():
    assert _pins_hold(Oracle)
    for mistake in ("swap_kv", "no_scale", "short_by_one", "own_layer", "head_mod"):
        assert not _pins_hold(lambda *a, m=mistake: _Mutant(m, *a)), f"the pins accept an oracle with '{mistake}'"


# ------------------------------------------------------------------ pre-fill rows (many query tokens at once)
def _causal_sdpa64(Q, K, V, pos, scale):
    """torch's library attention in fp64 with an explicit boolean mask: query row i sees keys t <= pos[i].
    Q [nq,Hq,D]; K,V [n,Hkv,D] of one sequence."""
    nq, Hq, D = Q.shape
    n, Hkv = K.shape[0], K.shape[1]
    G = Hq // Hkv
    q = Q.double().permute(1, 0, 2)[None]                                   # [1,Hq,nq,D]
    k = K.double().permute(1, 0, 2).repeat_interleave(G, 0)[None]           # [1,Hq,n,D]
    v = V.double().permute(1, 0, 2).repeat_interleave(G, 0)[None]
    mask = torch.arange(n)[None, :] <= pos.to(torch.int64)[:, None]         # [nq,n]
    out = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=mask[None, None], scale=scale)
    return out[0].permute(1, 0, 2)                                          # [nq,Hq,D]


@pytest.mark.parametrize("Hq,Hkv,D", [(4, 2, 32), (6, 2, 16), (4, 4, 64)])
def test_prefill_rows_equal_library_causal_attention(Hq, Hkv, D):
    """Whole prompt at once and a later chunk of it: library attention with a causal mask, on the source layer."""
    L, B, n = 3, 2, 29
    r = [0, 0, 2]
    o = Oracle(L, r, Hq, Hkv, D, B, n)
    store = _fill(o, L, B, n, Hkv, D, seed=17)
    for l in range(L):
        for b, (p0, p1) in enumerate([(0, 29), (11, 23)]):       # sequence 0: full prompt; sequence 1: a chunk
            pos = torch.arange(p0, p1)
            Q = _rand_bf16((pos.numel(), Hq, D), 300 + 10 * l + b)
            got = o.attn_rows(l, Q, torch.full_like(pos, b), pos, 0.21)
            want = _causal_sdpa64(Q, store[r[l]][0][b], store[r[l]][1][b], pos, 0.21)
            assert torch.allclose(got, want, rtol=1e-12, atol=1e-13)


def test_prefill_row_at_the_last_position_is_the_decode_step():
    """One row per sequence at pos = len-1 is Algorithm 2's decode attention."""
    L, B, n, Hq, Hkv, D = 2, 3, 17, 4, 2, 16
    o = Oracle(L, [0, 0], Hq, Hkv, D, B, n)
    _fill(o, L, B, n, Hkv, D, seed=19)
    lens = torch.tensor([17, 1, 9], dtype=torch.int32)
    Q = _rand_bf16((B, Hq, D), 77)
    a = o.attn_rows(1, Q, torch.arange(B), lens.to(torch.int64) - 1)
    assert torch.equal(a, o.decode_attn(1, Q, lens))


def test_prefill_first_token_sees_only_itself_and_rows_do_not_see_the_future():
    L, B, n, Hq, Hkv, D = 1, 1, 12, 4, 2, 16
    o = Oracle(L, [0], Hq, Hkv, D, B, n)
    store = _fill(o, L, B, n, Hkv, D, seed=23)
    pos = torch.arange(n)
    Q = _rand_bf16((n, Hq, D), 5)
    out = o.attn_rows(0, Q, torch.zeros(n, dtype=torch.int64), pos)
    assert torch.equal(out[0], store[0][1][0, 0].double().repeat_interleave(Hq // Hkv, 0))
    # overwrite the tokens after position 5: rows 0..5 must not move, rows 6.. must
    K2, V2 = _rand_bf16((n - 6, Hkv, D), 91), _rand_bf16((n - 6, Hkv, D), 92)
    o.append(0, K2, V2, torch.zeros(n - 6, dtype=torch.int64), torch.arange(6, n))
    out2 = o.attn_rows(0, Q, torch.zeros(n, dtype=torch.int64), pos)
    assert torch.equal(out2[:6], out[:6]) and not torch.equal(out2[6:], out[6:])


def test_prefill_brute_force_tiny():
    """Explicit weights without max-subtraction, a handful of rows."""
    L, B, n, Hq, Hkv, D = 2, 2, 5, 2, 1, 4
    o = Oracle(L, [0, 0], Hq, Hkv, D, B, n)
    store = _fill(o, L, B, n, Hkv, D, seed=29)
    q_seq = torch.tensor([0, 1, 1, 0])
    q_pos = torch.tensor([4, 0, 3, 2])
    Q = _rand_bf16((4, Hq, D), 31)
    got = o.attn_rows(1, Q, q_seq, q_pos, 0.5)
    for i in range(4):
        b, p = int(q_seq[i]), int(q_pos[i])
        for h in range(Hq):
            ws = [math.exp(0.5 * sum(float(Q[i, h, d]) * float(store[0][0][b, t, 0, d]) for d in range(D)))
                  for t in range(p + 1)]
            for d in range(D):
                want = sum(w * float(store[0][1][b, t, 0, d]) for t, w in enumerate(ws)) / sum(ws)
                assert abs(float(got[i, h, d]) - want) < 1e-12


# ------------------------------------------------------------------ training-time routing samplers (Section 3.2)
def test_rcla_map_cases_and_distribution():
    from oracle import rcla_map
    # hand cases: coin below p keeps the layer; otherwise floor(v * l) picks among the l layers before it
    assert rcla_map(0.5, [0.9, 0.9, 0.1, 0.9, 0.9], [0.0, 0.99, 0.5, 0.0, 0.999]) == [0, 0, 2, 0, 3]
    assert rcla_map(1.0, [0.3] * 6, [0.7] * 6) == list(range(6))          # p = 1: standard self-attention
    assert rcla_map(0.0, [0.0] * 4, [0.0, 0.0, 0.5, 0.9]) == [0, 0, 1, 2]   # p = 0: always a previous layer
    assert rcla_map(0.5, [1.0], [0.0]) is None                             # draws must lie in [0, 1)
    # distribution over many passes: P(self) = p for l >= 1, the choice is uniform on {0..l-1}
    g = torch.Generator().manual_seed(3)
    L, n, p = 9, 20000, 0.6
    self_count = torch.zeros(L)
    picks = torch.zeros(L, L)
    for _ in range(n // 100):
        U, V = torch.rand(100, L, generator=g, dtype=torch.float64), torch.rand(100, L, generator=g, dtype=torch.float64)
        for i in range(100):
            m = rcla_map(p, U[i].tolist(), V[i].tolist())
            for l, s in enumerate(m):
                assert 0 <= s <= l
                if s == l:
                    self_count[l] += 1
                else:
                    picks[l, s] += 1
    assert self_count[0] == n
    for l in range(1, L):
        # self includes d = 1 only (a cross pick is always < l)
        assert abs(self_count[l] / n - p) < 0.02
        cross = picks[l, :l]
        assert (cross / cross.sum() - 1.0 / l).abs().max() < 0.03


def test_rdcla_map_mixes_the_group_leader_and_the_layer_itself():
    from oracle import rdcla_map
    assert rdcla_map(4, 0.5, [0.9] * 8) == group_map(8, 4)                 # every coin says "shared": CLA@4
    assert rdcla_map(4, 0.5, [0.1] * 8) == list(range(8))                  # every coin says "own"
    assert rdcla_map(2, 0.6, [0.7, 0.7, 0.2, 0.9, 0.59, 0.61]) == [0, 0, 2, 2, 4, 4]
    assert rdcla_map(3, 0.6, [0.7, 0.2, 0.9, 0.2, 0.7, 0.61]) == [0, 1, 0, 3, 3, 3]


# ------------------------------------------------------------------ fp8 pages: the quantiser and attention over it
def test_e4m3_code_values_and_roundtrip():
    """All 254 finite codes: the value formula of the format (bias 7, 3 mantissa bits, subnormals, max 448),
    and torch's own float8_e4m3fn decoding of the same bits."""
    from oracle import e4m3_value
    codes = [c for c in range(256) if (c & 0x7f) != 0x7f]
    mine = torch.tensor([e4m3_value(c) for c in codes], dtype=torch.float64)
    theirs = torch.tensor(codes, dtype=torch.uint8).view(torch.float8_e4m3fn).double()
    assert torch.equal(mine, theirs)
    assert e4m3_value(0x7e) == 448.0 and e4m3_value(0x01) == 2.0 ** -9 and e4m3_value(0x08) == 2.0 ** -6
    assert e4m3_value(0xc5) == -(1 + 5 / 8) * 2.0


def test_e4m3_quantiser_matches_library_rounding_and_saturates():
    """Rows with amax = 448 have inv = 1, so codes = E4M3(x): torch's cast (round to nearest even) pins the
    rounding on random and on tie values; larger scales pin scale = amax/448 and saturation of the row maximum."""
    from oracle import quantize_e4m3
    g = torch.Generator().manual_seed(9)
    x = (torch.randn(64, 128, generator=g) * 40).clamp(-440, 440)
    x[:, 0] = 448.0                                                     # pins amax, so inv = 1 exactly
    ties = torch.tensor([2.0 ** -10, 1.5 * 2.0 ** -9, 2.5 * 2.0 ** -9, 17.0, 19.0, 0.0, -0.0, 2.0 ** -6 - 2.0 ** -10])
    x[0, 1:1 + ties.numel()] = ties
    xb = x.to(torch.bfloat16)
    codes, scales = quantize_e4m3(xb)
    want = xb.float().to(torch.float8_e4m3fn).view(torch.uint8)
    assert torch.equal(codes, want) and bool((scales == 1.0).all())
    # general scale: dequantised value within half a code step of the input, the row maximum maps to +-448
    y = (torch.randn(32, 64, generator=g) * 3).to(torch.bfloat16)
    c, s = quantize_e4m3(y)
    amax = y.float().abs().max(dim=1).values
    assert torch.equal(s, amax / 448.0)
    deq = c.view(torch.float8_e4m3fn).float() * s[:, None]
    assert bool(((deq - y.float()).abs() <= (amax[:, None] / 448.0) * 16.0 * 1.001 + 1e-6).all())    # coarsest step is 32 at the top binade
    top = y.float().abs().argmax(dim=1)
    assert bool((c[torch.arange(32), top] & 0x7f == 0x7e).all())
    z, sz = quantize_e4m3(torch.zeros(2, 16, dtype=torch.bfloat16))
    assert int(z.sum()) == 0 and bool((sz == 0).all())


def test_attention_over_fp8_layers_is_attention_over_the_dequantised_values():
    """A layer appended through the quantiser behaves exactly like a layer holding code x scale."""
    L, B, n, Hq, Hkv, D = 2, 2, 21, 4, 2, 32
    o = Oracle(L, [0, 0], Hq, Hkv, D, B, n)
    b_idx = torch.arange(B).repeat_interleave(n)
    t_idx = torch.arange(n).repeat(B)
    K = _rand_bf16((B * n, Hkv, D), 1, std=2.0)
    V = _rand_bf16((B * n, Hkv, D), 2, std=0.5)
    kc, vc, ks, vs = o.append_fp8(0, K, V, b_idx, t_idx)
    Kd = (kc.view(torch.float8_e4m3fn).double() * ks.double()[..., None]).view(B, n, Hkv, D)
    Vd = (vc.view(torch.float8_e4m3fn).double() * vs.double()[..., None]).view(B, n, Hkv, D)
    lens = torch.tensor([21, 8], dtype=torch.int32)
    Q = _rand_bf16((B, Hq, D), 3)
    G = Hq // Hkv
    got = o.decode_attn(1, Q, lens, 0.3)
    for b in range(B):
        nb = int(lens[b])
        q = Q[b].double()[None, :, None, :]
        k = Kd[b, :nb].permute(1, 0, 2).repeat_interleave(G, 0)[None]
        v = Vd[b, :nb].permute(1, 0, 2).repeat_interleave(G, 0)[None]
        want = torch.nn.functional.scaled_dot_product_attention(q, k, v, scale=0.3)[0, :, 0, :]
        assert torch.allclose(got[b], want, rtol=1e-12, atol=1e-13)
    # and it is close to, but not the same as, attention over the unquantised rows
    o2 = Oracle(L, [0, 0], Hq, Hkv, D, B, n)
    o2.append(0, K, V, b_idx, t_idx)
    ref = o2.decode_attn(1, Q, lens, 0.3)
    assert not torch.equal(got, ref) and (got - ref).abs().max() < 0.1
