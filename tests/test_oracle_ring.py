"""Pins of the oracle's circular buffer C(N, K) (Algorithm 1; Section 3.2)."""
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "splitmix64.txt")


def test_draw_matches_published_splitmix64_vectors(oracle):
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(rows) >= 8
    for seed, n, value in rows:
        assert oracle.draw_u64(int(seed), int(n)) == int(value)


def test_draw_matches_big_integer_arithmetic(oracle):
    mask = (1 << 64) - 1
    for seed in (0, 1, 0xDEADBEEF, mask):
        for n in (0, 1, 2, 1000, 2 ** 40):
            z = (seed + (n + 1) * 0x9E3779B97F4A7C15) & mask
            z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & mask
            z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & mask
            assert oracle.draw_u64(seed, n) == z ^ (z >> 31)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("N,K", [(1, 1), (2, 2), (16, 2), (32, 4), (4, 8)])
def test_every_batch_is_traversed_exactly_K_times(oracle, N, K, mode):
    ring = oracle.Ring(N, K, mode, seed=7)
    assert ring.sample()[0] == ring.EMPTY
    ids = {}
    for i in range(N):
        st, slot = ring.push()
        assert st == ring.OK and slot == i
        ids[slot] = i
    assert ring.push()[0] == ring.FULL
    assert ring.live() == N
    uses = np.zeros(N, int)
    seen_k = {s: [] for s in range(N)}
    for _ in range(N * K):
        st, slot, k = ring.sample()
        assert st == ring.OK
        uses[slot] += 1
        seen_k[slot].append(k)
    assert (uses == K).all()
    assert all(v == list(range(K)) for v in seen_k.values())
    assert ring.sample()[0] == ring.EMPTY
    assert ring.live() == 0


def test_steady_state_replaces_discarded_batches(oracle):
    N, K = 4, 3
    ring = oracle.Ring(N, K, 0, seed=11)
    pushed, sampled, next_id = 0, 0, 0
    owner = {}
    uses = {}
    for step in range(400):
        while True:
            st, slot = ring.push()
            if st != ring.OK:
                break
            owner[slot] = next_id
            uses[next_id] = 0
            next_id += 1
            pushed += 1
        st, slot, k = ring.sample()
        assert st == ring.OK
        assert k == uses[owner[slot]]
        uses[owner[slot]] += 1
        sampled += 1
    done = [u for i, u in uses.items() if i not in owner.values() or u == K]
    assert all(u <= K for u in uses.values())
    finished = [i for i, u in uses.items() if u == K]
    assert len(finished) >= 400 // K - N
    # samples = K x (finished batches) + partial traversals of the live ones
    assert sampled == sum(uses.values())
    assert pushed == len(uses)


def test_uniform_pick_follows_the_draw(oracle):
    N, K, seed = 5, 3, 99
    ring = oracle.Ring(N, K, 0, seed=seed)
    valid = [False] * N
    count = [0] * N
    for i in range(N):
        ring.push()
        valid[i] = True
    for n in range(N * K):
        live = [s for s in range(N) if valid[s]]
        u = oracle.draw_u64(seed, n)
        expect = live[(u * len(live)) >> 64]
        st, slot, k = ring.sample()
        assert (st, slot, k) == (0, expect, count[expect])
        count[expect] += 1
        if count[expect] == K:
            valid[expect] = False


def test_round_robin_order_and_push_cursor(oracle):
    ring = oracle.Ring(3, 2, 1, seed=0)
    for _ in range(3):
        ring.push()
    order = [ring.sample()[1] for _ in range(6)]
    assert order == [0, 1, 2, 0, 1, 2]
    assert ring.sample()[0] == ring.EMPTY
    # free slots are filled in ring order from the write cursor
    ring2 = oracle.Ring(3, 1, 1, seed=0)
    assert [ring2.push()[1] for _ in range(3)] == [0, 1, 2]
    assert ring2.sample()[1] == 0 and ring2.sample()[1] == 1
    assert ring2.push()[1] == 0 and ring2.push()[1] == 1
    assert ring2.push()[0] == ring2.FULL
    assert ring2.sample()[1] == 2
