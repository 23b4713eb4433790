"""CPU-side tests of the library: it loads, exports every declared symbol, validates its
arguments before touching CUDA, and its integer scheduling logic (Fade positions, effective
gates, K-list) agrees bit-for-bit with the oracle."""
import math
import os
import re
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2511_21089_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "mlpmoe.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(mlpmoe_[a-z0-9_]+)\s*\(", header))
    assert len(declared) >= 20
    for name in declared:
        assert hasattr(lib.lib, name), name
    assert declared == set(lib.SIGNATURES)
    assert lib.mlpmoe_status_string(0) == "ok"
    assert "keep" in lib.mlpmoe_status_string(lib.MLPMOE_ERR_EMPTY_KEEP_SET)


def test_create_rejects_bad_arguments_before_any_cuda_call(lib):
    import ctypes
    out = ctypes.c_void_p()
    fake = 0x1000  # never dereferenced: the checks below fail first

    def create(d, I, d_b, wg=fake, dtype=0, layout=0, max_tokens=16):
        arr = (ctypes.c_int64 * len(d_b))(*d_b)
        return lib.lib.mlpmoe_create(ctypes.byref(out), d, I, len(d_b), arr, wg, fake, fake, None, dtype, layout, max_tokens, None)

    assert create(64, 64, [32, 16]) == lib.MLPMOE_ERR_BAD_PARTITION          # does not sum to d_inter
    assert create(64, 64, [40, 24]) == lib.MLPMOE_ERR_BAD_PARTITION          # not multiples of 16
    assert create(64, 64, [64, 0]) == lib.MLPMOE_ERR_BAD_PARTITION
    assert create(64, 64, [32, 32], wg=None) == lib.MLPMOE_ERR_INVALID_ARG
    assert create(0, 64, [64]) == lib.MLPMOE_ERR_INVALID_ARG
    assert create(64, 64, [64], max_tokens=0) == lib.MLPMOE_ERR_INVALID_ARG
    assert create(64, 64, [64], dtype=7) == lib.MLPMOE_ERR_INVALID_ARG
    assert create(60, 64, [64]) == lib.MLPMOE_ERR_UNSUPPORTED                # d_model not a multiple of 8
    assert out.value is None
    # NULL handles are rejected everywhere, never dereferenced
    assert lib.lib.mlpmoe_forward(None, fake, fake, 1, None) == lib.MLPMOE_ERR_INVALID_ARG
    assert lib.lib.mlpmoe_fade(None, None, None) == lib.MLPMOE_ERR_INVALID_ARG
    assert lib.lib.mlpmoe_prune(None, None, 1, None) == lib.MLPMOE_ERR_INVALID_ARG
    assert lib.lib.mlpmoe_get_status(None) == lib.MLPMOE_ERR_INVALID_ARG
    lib.mlpmoe_destroy(None)


def test_fade_position_matches_oracle(lib):
    rng = np.random.default_rng(1)
    cases = [(0.0, 10), (0.5, 2), (0.9 * 31 / 32, 4096 * 448), (0.3, 1), (1e-300, 1 << 40), (0.999999999999, 1 << 40)]
    for _ in range(300):
        cases.append((float(rng.uniform(0, 1)), int(rng.integers(1, 1 << 36))))
    for k in range(1, 60):                      # products that land exactly on, or next to, an integer
        cases.append((k / 64.0, 64 * 977 + 1))
        cases.append((math.nextafter(k / 64.0, 0.0), 64 * 977 + 1))
    for s, m in cases:
        assert lib.mlpmoe_host_fade_position(s, m) == oracle.fade_position(s, m)[0], (s, m)
    for B in (4, 16, 32, 128):
        sched = oracle.fade_schedule(B)
        for b in range(B):
            for m in (896 * 304, 4096 * 448, 4096 * 64, 17):
                assert lib.mlpmoe_host_fade_position_default(b, B, m) == oracle.fade_position(sched[b], m)[0]
    import ctypes
    lo = ctypes.c_int64()
    assert lib.lib.mlpmoe_host_fade_position(1.0, 10, ctypes.byref(lo)) == lib.MLPMOE_ERR_BAD_SCHEDULE
    assert lib.lib.mlpmoe_host_fade_position(-0.1, 10, ctypes.byref(lo)) == lib.MLPMOE_ERR_BAD_SCHEDULE
    assert lib.lib.mlpmoe_host_fade_position(float("nan"), 10, ctypes.byref(lo)) == lib.MLPMOE_ERR_BAD_SCHEDULE


def test_prune_alpha_matches_oracle_bitwise(lib):
    rng = np.random.default_rng(2)
    for B in (4, 16, 64, 128):
        alpha = rng.uniform(0.8, 1.2, size=B).astype(np.float32)
        for n_drop in (0, 1, B // 4, B - 1):
            keep = synth.keep_set((5, B, n_drop), B, n_drop)
            for comp in (True, False):
                ours = lib.mlpmoe_host_prune_alpha(alpha.tolist(), keep, comp)
                ref = np.array(oracle.prune_alpha(alpha.astype(np.float64), keep, comp)).astype(np.float32)
                assert np.array_equal(ours.view(np.uint32), ref.view(np.uint32))
    with pytest.raises(lib.MlpmoeError) as e:
        lib.mlpmoe_host_prune_alpha([1.0, 1.0], [False, False])
    assert e.value.status == lib.MLPMOE_ERR_EMPTY_KEEP_SET
    # the paper's first-K rule, literally
    ours = lib.mlpmoe_host_prune_alpha([1.0] * 16, oracle.first_k_keep(16, 12))
    assert np.array_equal(ours[:12], np.full(12, np.float32(math.sqrt(16 / 12)))) and np.all(ours[12:] == 0)


def test_schedule_matches_oracle(lib):
    rng = np.random.default_rng(3)
    for trial in range(40):
        B = int(rng.integers(1, 9))
        d_b = [int(16 * rng.integers(1, 5)) for _ in range(B)]
        I = sum(d_b)
        alpha = rng.uniform(0.5, 1.5, size=B)
        alpha[rng.uniform(size=B) < 0.3] = 0.0
        p_dead = [0.0, 0.05, 0.5, 1.0][trial % 4]
        live = rng.uniform(size=I) >= p_dead
        # weights whose zero pattern gives exactly this liveness, through the three possible causes
        Wg, Wu, Wd = np.ones((2, I)), np.ones((2, I)), np.ones((I, 2))
        for j in np.nonzero(~live)[0]:
            (Wg[:, j], Wu[:, j], Wd[j, :])[int(rng.integers(0, 3))][...] = 0
        ref_b, ref_s = oracle.surviving_set(alpha, Wg, Wu, Wd, d_b)
        got_b, got_s, n_act = lib.mlpmoe_host_schedule(d_b, alpha.astype(np.float32).tolist(), live.tolist())
        assert got_b == ref_b and got_s == ref_s
        assert n_act == sum(l for _, l in ref_s)
    b, s, n = lib.mlpmoe_host_schedule([16, 32], [1.0, 1.0])
    assert (b, s, n) == ([0, 1], [(0, 16), (16, 32)], 48)


def test_synth_generators():
    import torch
    a = synth.normal_f32((1, 2, 3, 4), (3, 1 << 20), 0.02, threads=1)
    b = synth.normal_f32((1, 2, 3, 4), (3, 1 << 20), 0.02, threads=8)
    assert np.array_equal(a, b)                                   # independent of the thread count
    assert abs(float(a.std()) - 0.02) < 2e-4 and abs(float(a.mean())) < 1e-4
    assert not np.array_equal(a, synth.normal_f32((1, 2, 3, 5), (3, 1 << 20), 0.02))
    bits = synth.f32_to_bf16_bits(a[0, :4096])
    ref = torch.from_numpy(a[0, :4096].copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    assert np.array_equal(synth.bf16_bits_to_f32(bits), torch.from_numpy(a[0, :4096].copy()).to(torch.bfloat16).float().numpy())
    for B in (4, 8, 16, 32, 64, 128):
        p = synth.random_partition((9, B), 14336, B, 64)
        assert len(p) == B and sum(p) == 14336 and all(w > 0 and w % 64 == 0 for w in p)
        assert p == synth.random_partition((9, B), 14336, B, 64)
    assert len(set(synth.random_partition((9, 16), 14336, 16, 64))) > 1
    assert synth.equal_partition(4864, 16) == [304] * 16
    k = synth.keep_set((7,), 16, 4)
    assert sum(k) == 12 and k == synth.keep_set((7,), 16, 4)
    assert [synth.n_drop_for_ratio(B, r) for B in (4, 32, 128) for r in (0.0, 0.1, 0.2, 0.4)] == \
        [0, 0, 1, 2, 0, 3, 6, 13, 0, 13, 26, 51]


@pytest.mark.parametrize("n,d,Ipad,bn,ks", [(4096, 896, 3712, 224, 1), (4096, 896, 3712, 224, 3), (300, 320, 512, 128, 4),
                                            (8192, 4096, 14336, 256, 1), (2048, 4096, 11520, 256, 2),
                                            (16384, 4096, 14336, 256, 1), (129, 64, 128, 64, 1)])
def test_tile_schedule_is_complete_and_cannot_deadlock(lib, n, d, Ipad, bn, ks):
    """Every tile exactly once; and whatever the tiles' real durations turn out to be, running the
    per-pair sequences with 'a down tile waits for all gate|up tiles of its token block' finishes."""
    lists = lib.mlpmoe_host_tile_schedule(n, d, Ipad, bn, ks, 148)
    m_pairs, n1, n2 = (n + 255) // 256, Ipad // 128, ks * ((d + bn - 1) // bn)
    flat = [t for l in lists for t in l]
    assert len(flat) == len(set(flat)) == m_pairs * (n1 + n2)
    assert set(flat) == {(0, nb, m) for nb in range(n1) for m in range(m_pairs)} | {(1, nb, m) for nb in range(n2) for m in range(m_pairs)}
    rng = np.random.default_rng(n)
    for trial in range(3):
        dur = {t: float(rng.uniform(0.1, 10.0)) for t in flat}            # arbitrary durations
        pos = [0] * len(lists)
        clock = [0.0] * len(lists)
        left = {m: n1 for m in range(m_pairs)}
        done_at = {m: 0.0 for m in range(m_pairs)}
        remaining = len(flat)
        while remaining:
            progressed = False
            # run the pair with the smallest clock whose next tile is runnable
            order = sorted(range(len(lists)), key=lambda c: clock[c])
            for c in order:
                if pos[c] >= len(lists[c]):
                    continue
                t = lists[c][pos[c]]
                if t[0] == 1 and left[t[2]] > 0:
                    continue                                           # blocked: its token block is not complete
                start = max(clock[c], done_at[t[2]]) if t[0] == 1 else clock[c]
                clock[c] = start + dur[t]
                if t[0] == 0:
                    left[t[2]] -= 1
                    done_at[t[2]] = max(done_at[t[2]], clock[c])
                pos[c] += 1
                remaining -= 1
                progressed = True
                break
            assert progressed, "every pair is blocked on a down tile: the schedule can deadlock"
    # balance under the cost model: no pair gets more than its share plus one large tile
    loads = [sum((Ipad // 64) * max(2 * bn, (16384 + bn * 64) // 50) // ks if t[0] else ((d + 63) // 64) * 655 for t in l) for l in lists]
    if m_pairs * (n1 + n2) >= 4 * 74:
        assert max(loads) <= 1.35 * (sum(loads) / len(loads))


@pytest.mark.parametrize("n,d,Ipads,kss,bn", [(4096, 896, [3712, 3712, 4864], [3, 3, 2], 224), (300, 128, [256, 128], [1, 1], 128),
                                              (2048, 4096, [14336, 11520], [1, 1], 256), (257, 896, [3712], [4], 224)])
def test_stack_schedule_is_complete_and_cannot_deadlock(lib, n, d, Ipads, kss, bn):
    """Every item of every layer exactly once; and whatever the items' real durations turn out to be,
    running the sequences (per pair one of GEMM items and, independently, one of norm parts) under
    the kernel's three waiting rules finishes: a norm part waits for all down items of its token
    block in the previous layer, a gate|up tile for all norm parts of its block, a down item for
    all gate|up tiles of its block."""
    gemm, norm = lib.mlpmoe_host_stack_schedule(n, d, Ipads, kss, bn, 148)
    assert all(t[0] != 2 for lst in gemm for t in lst) and all(t[0] == 2 for lst in norm for t in lst)
    lists = gemm + norm
    m_pairs, L = (n + 255) // 256, len(Ipads)
    n2 = (d + bn - 1) // bn
    want = set()
    for l in range(L):
        for m in range(m_pairs):
            want |= {(2, part, m, l) for part in range(16)}
            want |= {(0, nb, m, l) for nb in range(Ipads[l] // 128)}
            want |= {(1, nb, m, l) for nb in range(n2 * kss[l])}
    flat = [t for lst in lists for t in lst]
    assert len(flat) == len(set(flat)) and set(flat) == want
    need = {}                      # (kind it waits on, block, layer) -> arrivals needed
    for l in range(L):
        for m in range(m_pairs):
            need[(2, m, l)] = 16
            need[(0, m, l)] = Ipads[l] // 128
            need[(1, m, l)] = n2 * kss[l]

    def blocked(t, have):
        typ, _, m, l = t
        if typ == 2:
            return l > 0 and have.get((1, m, l - 1), 0) < need[(1, m, l - 1)]
        if typ == 0:
            return have.get((2, m, l), 0) < need[(2, m, l)]
        return have.get((0, m, l), 0) < need[(0, m, l)]

    rng = np.random.default_rng(n)
    for trial in range(2):
        # the pair to advance is drawn at random among the runnable ones: any interleaving must finish
        pos = [0] * len(lists)
        have = {}
        remaining = len(flat)
        while remaining:
            runnable = [c for c in range(len(lists)) if pos[c] < len(lists[c]) and not blocked(lists[c][pos[c]], have)]
            assert runnable, "every pair is blocked: the schedule can deadlock"
            for c in rng.permutation(runnable)[: max(1, len(runnable) // 2)]:
                t = lists[c][pos[c]]
                have[(t[0], t[2], t[3])] = have.get((t[0], t[2], t[3]), 0) + 1
                pos[c] += 1
                remaining -= 1
    counts = [len(lst) for lst in gemm]
    if len(flat) >= 8 * 74:
        assert max(counts) <= 1.5 * (sum(counts) / len(counts)) + 4


@pytest.mark.parametrize("blocks,d,Ipads,bn", [([0] * 8 + [1] * 3 + [3] * 9, 4096, [512, 512, 384, 512], 256),
                                                ([2, 0, 0, 1], 320, [128, 256, 128], 160),
                                                (sum(([b] * 8 for b in range(32)), []), 4096, [512] * 32, 256), ([], 256, [128], 128)])
def test_group_schedule_is_complete_and_cannot_deadlock(lib, blocks, d, Ipads, bn):
    """The one grouped launch of the routed forward: every block has exactly its branch's gate|up tiles and its down
    items, once; a down item waits for all gate|up tiles of its block and nothing else waits; whatever the items' real
    durations, running the pairs' sequences under that rule finishes; the items are spread evenly."""
    lists = lib.mlpmoe_host_group_schedule(blocks, d, Ipads, bn, 148)
    n2 = (d + bn - 1) // bn
    want = set()
    for r, b in enumerate(blocks):
        want |= {(0, nb, r, b) for nb in range(Ipads[b] // 128)}
        want |= {(1, nb, r, b) for nb in range(n2)}
    flat = [t for lst in lists for t in lst]
    assert len(flat) == len(set(flat)) and set(flat) == want
    rng = np.random.default_rng(len(blocks))
    for trial in range(2):
        pos = [0] * len(lists)
        tiles_done = {}
        remaining = len(flat)
        while remaining:
            runnable = [c for c in range(len(lists)) if pos[c] < len(lists[c]) and
                        (lists[c][pos[c]][0] == 0 or tiles_done.get(lists[c][pos[c]][2], 0) == Ipads[lists[c][pos[c]][3]] // 128)]
            assert runnable, "every pair is blocked: the schedule can deadlock"
            for c in rng.permutation(runnable)[: max(1, len(runnable) // 2)]:
                t = lists[c][pos[c]]
                if t[0] == 0:
                    tiles_done[t[2]] = tiles_done.get(t[2], 0) + 1
                pos[c] += 1
                remaining -= 1
    if len(flat) >= 8 * 74:
        cost = [sum(64 * 512 if t[0] == 0 else Ipads[t[3]] // 64 * 2 * bn for t in lst) for lst in lists]
        assert max(cost) <= 1.1 * (sum(cost) / len(cost)) + 64 * 512
