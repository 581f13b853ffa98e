"""Host logic: the C-ABI library loads without a GPU, exports every declared
symbol, validates its arguments, and the planner's tile map agrees with the
oracle's dense Algorithm-3 mask tile by tile."""
import os
import re

import numpy as np
import pytest

from oracle import psa_oracle as orc
from paper_2410_20305_b200 import binding as B
from paper_2410_20305_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TILE = 128


def test_library_exports_every_declared_symbol():
    lib = B.load_library()
    header = open(os.path.join(ROOT, "include", "psa.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(psa_[a-z0-9_]+|dpo_lo[a-z0-9_]*|simpo_[a-z_]+|orpo_[a-z_]+)\s*\(", header))
    declared.discard("psa_status_t")
    assert declared, "no declarations found"
    assert set(B.EXPORTED_SYMBOLS) >= declared
    for name in declared:
        assert hasattr(lib, name), name


def _plan(pack, **kw):
    return B.psa_plan(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len,
                      pack.n_q_heads, pack.n_kv_heads, pack.head_dim, host_only=True, **kw)


def _check_against_dense_mask(pack):
    plan = _plan(pack)
    mask = orc.packed_mask(pack.cu_seqlens, pack.prefix_len, pack.chosen_len, pack.rejected_len)
    T = pack.total_tokens
    assert plan.total_tokens == T
    assert plan.useful_pairs == int(mask.sum())
    f_tiles, f_ent = plan.export(0)
    b_tiles, b_ent = plan.export(1)
    sample_of = {int(pack.cu_seqlens[s]): s for s in range(pack.n_samples)}

    def dense_class(ds, length, i, j, bwd):
        """0 dropped / 1 full / 2 partial, from the dense mask, tile (i, j) of the sample at ds."""
        q0, k0 = ds + i * TILE, ds + j * TILE
        q1, k1 = min(q0 + TILE, ds + length), min(k0 + TILE, ds + length)
        sub = mask[q0:q1, k0:k1]
        if not sub.any():
            return 0
        full = sub.all() and (k1 - k0 == TILE) and (not bwd or q1 - q0 == TILE)
        return 1 if full else 2

    fwd_set, n_live, n_partial = {}, 0, 0
    precise_of = {}
    seen_tiles = set()
    for row0, ds, local0, length, cs, rs, off, cnt in f_tiles:
        s = sample_of[int(ds)]
        assert length == pack.cu_seqlens[s + 1] - ds and cs == pack.prefix_len[s] and rs == cs + pack.chosen_len[s]
        assert row0 == ds + local0 and local0 % TILE == 0 and local0 < length
        i = local0 // TILE
        seen_tiles.add((s, i))
        listed = {int(e) >> 2: int(e) & 1 for e in f_ent[off:off + cnt]}
        precise = {int(e) >> 2: (int(e) >> 1) & 1 for e in f_ent[off:off + cnt]}
        assert len(listed) == cnt
        assert sorted(listed) == [int(e) >> 2 for e in f_ent[off:off + cnt]], "key tiles must ascend"
        q_lo, q_hi = int(ds) + i * TILE, min(int(ds) + i * TILE + TILE, int(ds) + int(length))
        few_keys = bool((mask[q_lo:q_hi].sum(axis=1) < TILE).any())
        assert all(p == int(few_keys) for p in precise.values()), (s, i, few_keys)
        precise_of[(s, i)] = int(few_keys)
        for j in range((length + TILE - 1) // TILE):
            c = dense_class(int(ds), int(length), i, j, False)
            if c == 0:
                assert j not in listed, (s, i, j)
            else:
                assert j in listed, (s, i, j)
                # a tile flagged full must truly need no mask; a truly partial one must be flagged
                if c == 2:
                    assert listed[j] == 1, (s, i, j)
                n_live += 1
                n_partial += listed[j]
                fwd_set[(s, i, j)] = listed[j]
    n_tiles = sum((int(pack.cu_seqlens[s + 1] - pack.cu_seqlens[s]) + TILE - 1) // TILE for s in range(pack.n_samples))
    assert len(seen_tiles) == len(f_tiles) == n_tiles
    assert plan.live_tiles == n_live and plan.partial_tiles == n_partial
    # longest-first order
    assert list(f_tiles[:, 7]) == sorted(f_tiles[:, 7], reverse=True)
    assert list(b_tiles[:, 7]) == sorted(b_tiles[:, 7], reverse=True)

    bwd_set = {}
    for row0, ds, local0, length, cs, rs, off, cnt in b_tiles:
        s = sample_of[int(ds)]
        j = local0 // TILE
        for e in b_ent[off:off + cnt]:
            i = int(e) >> 2
            c = dense_class(int(ds), int(length), i, j, True)
            assert c != 0
            if c == 2:
                assert int(e) & 1 == 1, (s, i, j)
            bwd_set[(s, i, j)] = int(e) & 1
            assert (int(e) >> 1) & 1 == precise_of[(s, i)], (s, i, j)
    assert set(bwd_set) == set(fwd_set), "forward and transposed maps hold the same tiles"
    plan.close()


def test_tiny_config_tile_map():
    _check_against_dense_mask(wl.config_pack(0))


@pytest.mark.parametrize("seed", range(6))
def test_random_packs_tile_map(seed):
    _check_against_dense_mask(wl.random_pack(100 + seed, 4, 400, 4, 2, 64))


def test_boundaries_on_and_off_tile_edges():
    lengths = [(128, 128, 128), (256, 0, 128), (0, 128, 256), (127, 129, 1), (129, 127, 255), (1, 0, 0),
               (384, 1, 1), (100, 300, 300)]
    _check_against_dense_mask(wl.pack_from_lengths("edges", lengths, 2, 1, 64))


def test_short_many_config_tile_map():
    _check_against_dense_mask(wl.config_pack(4))


def test_stats_of_bench_configs():
    for idx in (1, 2, 3):
        pack = wl.config_pack(idx)
        plan = _plan(pack)
        assert plan.useful_pairs == orc.useful_pairs(pack.prefix_len, pack.chosen_len, pack.rejected_len)
        assert plan.bwd_workspace_bytes >= pack.total_tokens * 32 * 128 * 4
        assert 0 < plan.partial_tiles < plan.live_tiles
        plan.close()


def test_argument_validation():
    ok = dict(n_q_heads=4, n_kv_heads=2, head_dim=64, host_only=True)
    with pytest.raises(B.PsaError) as e:
        B.psa_plan([0, 10], [4], [3], [4], **ok)           # 4+3+4 != 10
    assert e.value.code == 2
    with pytest.raises(B.PsaError) as e:
        B.psa_plan([1, 11], [4], [3], [3], **ok)           # cu_seqlens[0] != 0
    assert e.value.code == 2
    with pytest.raises(B.PsaError) as e:
        B.psa_plan([0, 10], [-1], [8], [3], **ok)
    assert e.value.code == 1
    with pytest.raises(B.PsaError) as e:
        B.psa_plan([0, 10], [4], [3], [3], 4, 3, 64, host_only=True)   # Hq % Hkv
    assert e.value.code == 3
    with pytest.raises(B.PsaError) as e:
        B.psa_plan([0, 10], [4], [3], [3], 4, 2, 96, host_only=True)   # head_dim
    assert e.value.code == 3
    empty = B.psa_plan([0], [], [], [], **ok)               # no samples: a valid, empty plan
    assert empty.total_tokens == 0 and empty.live_tiles == 0
    zero_len = B.psa_plan([0, 0, 5], [0, 2], [0, 2], [0, 1], **ok)   # a zero-length sample is skipped
    assert zero_len.export(0)[0].shape[0] == 1


def test_host_only_plan_is_refused_by_the_kernels():
    plan = B.psa_plan([0, 10], [4], [3], [3], 4, 2, 64, host_only=True)
    lib = B.load_library()
    assert lib.psa_fwd(plan._h, 16, 16, 16, 16, 16, None, None) == 1
