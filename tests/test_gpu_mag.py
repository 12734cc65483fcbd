"""Parity of csd_mag_draft with the oracle (bit-exact), including tables small enough to force
hash collisions."""
import numpy as np
import pytest

import workloads
from gpu_util import require_gpu, to_dev_i32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    require_gpu()
    from paper_2312_11462_b200 import binding
    return binding


def test_random_cases_and_forced_collisions(b, orc):
    rng = np.random.default_rng(0)
    for trial in range(120):
        V = int(rng.choice([3, 5, 50, 4096]))
        L = int(rng.integers(1, 200))
        T = int(rng.integers(1, 60))
        n = int(rng.integers(1, 17))
        order = int(rng.choice([1, 2, 3, 16, 32]))
        hay = rng.integers(0, V, size=L).astype(np.int32)
        if trial % 2 == 0:
            hay = workloads.make_repetitive_prompt(V, L, int(rng.integers(1 << 30)))
        seq = rng.integers(0, V, size=T).astype(np.int32)
        if trial % 3 == 0 and T >= L:
            seq[T - L:] = hay
        if trial % 3 == 1 and L > 8:
            s = int(rng.integers(0, L - 4)); w = min(T, L - s - 1, 6)
            if w > 0:
                seq[T - w:] = hay[s:s + w]
        nxt = rng.integers(0, V, size=V).astype(np.int32)
        want = orc.mag_draft(hay, nxt, seq, n, order)
        grams = sum(max(L - o, 0) for o in range(1, order + 1))
        tight = 64
        while tight < grams + 1:
            tight *= 2
        for slots in (0, tight):                 # default table, and the smallest legal one
            g = b.Mag(to_dev_i32(hay), to_dev_i32(nxt), order, slots)
            got = g.csd_mag_draft(to_dev_i32(seq), n).cpu().numpy()
            assert got.tolist() == want.tolist(), (trial, slots, hay, seq, n, order)
            g.close()
    assert b.csd_device_status() == 0


def test_workload_shapes(b, orc):
    for L, V in ((32, 4096), (128, 32000), (256, 32128), (2048, 32000)):
        hay = workloads.make_prompt(V, L, seed=L)
        nxt = workloads.bigram_table(hay, V, seed=1)
        g = b.Mag(to_dev_i32(hay), to_dev_i32(nxt), 16)
        rng = np.random.default_rng(L)
        for _ in range(10):
            cut = int(rng.integers(2, L))
            seq = np.concatenate([hay, hay[cut - 2:cut], rng.integers(0, V, size=int(rng.integers(0, 2)))]).astype(np.int32)
            n = int(rng.choice([1, 4, 10, 16]))
            got = g.csd_mag_draft(to_dev_i32(seq), n).cpu().numpy()
            assert got.tolist() == orc.mag_draft(hay, nxt, seq, n, 16).tolist()
        g.close()


def test_in_place_append_and_errors(b, orc):
    import torch
    hay = workloads.make_repetitive_prompt(30, 64, seed=3)
    nxt = workloads.bigram_table(hay, 30, seed=1)
    g = b.Mag(to_dev_i32(hay), to_dev_i32(nxt), 16)
    buf = torch.zeros(100, dtype=torch.int32, device="cuda")
    buf[:64] = to_dev_i32(hay)
    from paper_2312_11462_b200.binding import lib, _check, _ptr, _stream
    _check("csd_mag_draft", lib.csd_mag_draft(g.h, _ptr(buf), 64, 10, buf.data_ptr() + 64 * 4, _stream()))
    assert buf[64:74].cpu().numpy().tolist() == orc.mag_draft(hay, nxt, hay, 10, 16).tolist()
    assert lib.csd_mag_draft(g.h, _ptr(buf), 0, 10, _ptr(buf), _stream()) == 1
    assert lib.csd_mag_draft(g.h, _ptr(buf), 5, 65, _ptr(buf), _stream()) == 1
    with pytest.raises(b.CsdError):
        b.Mag(to_dev_i32(hay), to_dev_i32(nxt), 16, 64)      # table too small for the n-grams


def test_dynamic_haystack_against_the_oracle(b, orc):
    # haystack = static part followed by the generated part of the sequence; the oracle searches the
    # joined text.  Small vocabularies and repeated phrases make matches that lie inside the static
    # part, straddle its end, lie inside the generation, or whose follower is the first generated token.
    rng = np.random.default_rng(1)
    for trial in range(150):
        V = int(rng.choice([3, 5, 50]))
        L = int(rng.integers(0, 80))
        P = int(rng.integers(1, 20))                       # tokens of the sequence before the generation
        G = int(rng.integers(0, 70))                       # generated tokens
        n = int(rng.integers(1, 17))
        order = int(rng.choice([1, 2, 3, 16, 32]))
        hay = (workloads.make_repetitive_prompt(V, L, int(rng.integers(1 << 30))) if trial % 2 == 0 and L > 0
               else rng.integers(0, V, size=L).astype(np.int32))
        seq = rng.integers(0, V, size=P + G).astype(np.int32)
        if trial % 3 == 0 and G > 12:                      # a phrase repeated inside the generation
            w = int(rng.integers(2, 6))
            seq[P + G - w:] = seq[P + 2:P + 2 + w]
        if trial % 3 == 1 and L > 4 and G >= 3:            # the generation continues the static part's end
            seq[-2:] = hay[-2:]
        nxt = rng.integers(0, V, size=V).astype(np.int32)
        joined = np.concatenate([hay, seq[P:]]).astype(np.int32)
        want = orc.mag_draft(joined, nxt, seq, n, order)
        g = b.Mag(to_dev_i32(hay) if L > 0 else to_dev_i32([0])[:0], to_dev_i32(nxt), order)
        got = g.csd_mag_draft_dynamic(to_dev_i32(seq), P, n).cpu().numpy()
        assert got.tolist() == want.tolist(), (trial, hay, seq, P, n, order)
        # nothing generated yet: the static search
        got0 = g.csd_mag_draft_dynamic(to_dev_i32(seq[:P]), P, n).cpu().numpy()
        assert got0.tolist() == orc.mag_draft(hay, nxt, seq[:P], n, order).tolist()
        g.close()
    assert b.csd_device_status() == 0
