"""Host-side checks of the C-ABI library that need no GPU: it loads, exports what the header
declares, parses policy blobs like the oracle does, sizes caches, and partitions decode work so
that every page is processed exactly once."""
import ctypes as C
import os
import re
import subprocess

import numpy as np
import pytest

from pask_workloads import configs as WC
from pask_workloads import policy as WP

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def pask():
    subprocess.run(["python", os.path.join(ROOT, "paper_2608_28276_b200", "build.py"), "--if-stale"], check=True,
                   capture_output=True)
    import paper_2608_28276_b200 as P
    return P


def test_library_exports_every_declared_symbol(pask):
    header = open(os.path.join(ROOT, "include", "pask.h")).read()
    declared = set(re.findall(r"\b(pask_[a-z0-9_]+)\s*\(", header))
    declared -= {"pask_budget_state_t"}
    assert declared == set(pask.EXPORTS), declared ^ set(pask.EXPORTS)
    lib = C.CDLL(pask.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_layouts_match_header(pask):
    assert C.sizeof(pask.BudgetState) == 4 * 8 * 8 + 4 * 8 + 4 * 4 + 5 * 8
    assert C.sizeof(pask.CacheDesc) == 48


def test_policy_blob_parsing_agrees_with_oracle(pask, oracle):
    for cfg in (WC.TINY, WC.QWEN3_4B_1LAYER):
        w = WC.build(cfg)
        h = pask.pask_load_policy(w.blob)
        o = oracle.Policy(w.blob)
        for z in range(w.policy.n_tags):
            for c in range(w.policy.n_groups):
                assert pask.pask_policy_action(h, z, c) == o.action(z, c) == max(w.policy.a0[z, c], w.policy.a_floor[z, c])
        assert pask.pask_policy_action(h, w.policy.n_tags, 0) == -1
        pask.pask_free_policy(h)


def test_version_2_blobs(pask, oracle):
    # critical-state flags and the reserve shift ride behind gamma; both loaders take and refuse the same blobs
    w = WC.build(WC.scaled(WC.QWEN3_4B_1LAYER, batch=1, prompt_len=32, gen_len=32))
    good = w.dynamic_blob()
    assert good[4] == 2
    pask.pask_free_policy(pask.pask_load_policy(good))
    oracle.Policy(good)
    n_states = int.from_bytes(good[20:24], "little")
    crit_at = len(good) - ((n_states + 3) // 4) * 4
    bads = [good[:-4], good + b"\0\0\0\0"]
    b = bytearray(good); b[crit_at] = 2; bads.append(bytes(b))                 # a flag that is not 0 or 1
    b = bytearray(good); b[crit_at - 4] = 17; bads.append(bytes(b))            # gamma_shift > 16
    b = bytearray(good); b[40 + 4 + 4:40 + 4 + 8] = b"\x00\x00\xc0\x7f"; bads.append(bytes(b))   # a NaN score
    for blob in bads:
        with pytest.raises(pask.PaskError) as e:
            pask.pask_load_policy(blob)
        assert e.value.status == pask.ERR_BAD_POLICY
        with pytest.raises(ValueError):
            oracle.Policy(blob)


def test_bad_blobs_and_arguments_are_refused(pask):
    good = WC.build(WC.TINY).blob
    bads = [good[:-1], good + b"\0", b"XASK" + good[4:], good[:4] + b"\2\0\0\0" + good[8:], b"PASK", b""]
    broken = bytearray(good); broken[40 + 4] = 3; bads.append(bytes(broken))           # action out of range
    broken = bytearray(good); broken[28] = 1; bads.append(bytes(broken))               # recent window not a multiple of 16
    broken = bytearray(good); broken[29] = 2; bads.append(bytes(broken))               # recent window too large (512)
    broken = bytearray(good); broken[32] = 6; bads.append(bytes(broken))               # low_bits none of 2, 4, 8
    broken = bytearray(good); broken[40] = 9; bads.append(bytes(broken))               # layer group out of range
    for b in bads:
        with pytest.raises(pask.PaskError) as e:
            pask.pask_load_policy(b)
        assert e.value.status == pask.ERR_BAD_POLICY
    d = pask.CacheDesc(1, 8, 2, 128, 16, 4, 1024, 1024, 8, 8)
    assert pask.pask_cache_sizes(d).high_page_bytes == 2 * 8192
    assert pask.pask_cache_sizes(d).low_page_bytes == 2 * 2304
    for bad in (pask.CacheDesc(1, 8, 2, 64, 16, 4, 1024, 1024, 8, 8), pask.CacheDesc(1, 8, 2, 128, 32, 4, 1024, 1024, 8, 8),
                pask.CacheDesc(1, 6, 2, 128, 16, 4, 1024, 1024, 8, 8), pask.CacheDesc(1, 12, 3, 128, 16, 4, 1024, 1024, 8, 8)):
        with pytest.raises(pask.PaskError) as e:
            pask.pask_cache_sizes(bad)
        assert e.value.status == pask.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(pask.PaskError) as e:
        pask.pask_cache_sizes(pask.CacheDesc(0, 8, 2, 128, 16, 4, 1024, 1024, 8, 8))
    assert e.value.status == pask.ERR_INVALID_ARG
    assert pask.pask_status_string(pask.ERR_POOL_EXHAUSTED) == "page pool exhausted"
    assert pask.pask_status_string(pask.ERR_NO_MEMORY) == "out of host memory"


def test_decode_partition_covers_every_page_exactly_once(pask):
    rng = np.random.default_rng(3)
    cases = [([5], [0], 4), ([0], [7], 3), ([0, 0, 3], [0, 2, 0], 8), ([1], [1], 296),
             ([513] * 8, [0] * 8, 296), ([100, 0, 3000, 1, 0, 40], [900, 0, 100, 0, 2, 7], 296), ([2000, 1], [0, 0], 32)]
    for _ in range(30):
        n = int(rng.integers(1, 40))
        cases.append((rng.integers(0, 60, n), rng.integers(0, 90, n), int(rng.choice([1, 2, 7, 64, 296]))))
    for ph, pl, g in cases:
        ph, pl = np.asarray(ph, np.uint32), np.asarray(pl, np.uint32)
        r = pask.pask_debug_partition(ph, pl, g).astype(np.int64)
        cost = np.zeros(g)
        for s in range(len(ph)):
            is_high, idx = pask.pask_debug_page_order(int(ph[s]), int(pl[s]))
            # the order visits every HIGH page and every LOW page once, each stream in ascending order
            assert np.array_equal(idx[is_high], np.arange(ph[s])) and np.array_equal(idx[~is_high], np.arange(pl[s]))
            # and interleaves them evenly: any prefix holds its proportional share of HIGH pages
            if len(idx):
                seen_high = np.cumsum(is_high)
                want = np.arange(1, len(idx) + 1) * float(ph[s]) / len(idx)
                assert np.abs(seen_high - want).max() <= 1.0
            seen = np.zeros(len(idx), np.int64)
            last_end = 0
            for b in range(g):
                a, e = r[b, s]
                assert a <= e
                if e > a:
                    assert a == last_end          # contiguous, in CTA order
                    last_end = e
                seen[a:e] += 1
                cost[b] += 32 * is_high[a:e].sum() + 9 * (~is_high[a:e]).sum()
            assert np.all(seen == 1)
        total = float(32 * ph.sum() + 9 * pl.sum())
        assert cost.sum() == total
        if 16 * len(ph) <= g:
            # a small batch: every non-empty sequence has whole CTAs of its own, one plus its share of the others, so a
            # CTA streams at most g / (g - sequences) of an even share plus about a page of each kind
            owners = [set(np.nonzero(r[:, s, 1] > r[:, s, 0])[0]) for s in range(len(ph))]
            for s in range(len(ph)):
                assert (len(owners[s]) > 0) == (ph[s] + pl[s] > 0)
                assert all(owners[s].isdisjoint(owners[t]) for t in range(s))
                if ph[s] + pl[s] >= g:      # enough pages to give every CTA some: the count is one plus the rounded share
                    n_ne = int(np.count_nonzero(ph + pl))
                    assert abs(len(owners[s]) - 1 - (g - n_ne) * (32.0 * ph[s] + 9.0 * pl[s]) / total) <= 1.0
            assert cost.max() <= total / (g - len(ph)) + 2 * (32 + 9) + 1e-9
        else:
            # balance: no CTA streams more than its share plus about one page of each kind per cut
            assert cost.max() <= total / g + 2 * (32 + 9) + 1e-9
