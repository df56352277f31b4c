"""Circular buffer and gathers on the GPU against the oracle's ring: bit-exact."""
import numpy as np
import pytest
import torch

import impact_inputs as ii

pytestmark = pytest.mark.gpu


def _fields(cfg_idx, seed):
    cfg, b = ii.make_config(cfg_idx, seed=seed)
    names = ["actions", "rewards", "discounts", "worker_logp", "target_logits"]
    return cfg, [np.ascontiguousarray(b[n]) for n in names], b


def _drive(oracle, N, K, mode, seed, field_arrays_fn, steps, gather=False, host_src=False):
    """Runs the same push/sample script on both rings; returns nothing, asserts equality."""
    import paper_1912_00167_b200 as ip
    first = field_arrays_fn(0)
    fb = [a.nbytes for a in first]
    ring = ip.ImpactBuffer(N, K, fb, seed=seed, sample_mode=mode)
    ref = oracle.Ring(N, K, mode, seed=seed)
    payload = {}
    next_id = 0
    rng = np.random.default_rng(seed)
    dsts = [torch.empty(a.nbytes, dtype=torch.uint8, device="cuda") for a in first]
    for step in range(steps):
        if rng.random() < 0.45:
            arrays = field_arrays_fn(next_id)
            src = [torch.from_numpy(a) if host_src else torch.from_numpy(a).cuda() for a in arrays]
            if host_src:
                src = [s.pin_memory() for s in src]
            slot = ring.push(src)
            st, rslot = ref.push()
            if st == ref.FULL:
                assert slot is None
            else:
                assert slot == rslot
                payload[slot] = arrays
                next_id += 1
        else:
            got = ring.sample(gather_dst=dsts if gather else None)
            st, rslot, rk = ref.sample()
            if st == ref.EMPTY:
                assert got is None
                continue
            assert got == (rslot, rk)
            torch.cuda.synchronize()
            for f, a in enumerate(payload[rslot]):
                view = ring.slot_view(rslot, f, torch.uint8, (a.nbytes,))
                assert bytes(view.cpu().numpy()) == a.tobytes()
                if gather:
                    assert bytes(dsts[f].cpu().numpy()) == a.tobytes()
        assert ring.live() == ref.live()
    ring.close()


@pytest.mark.parametrize("cfg_idx,mode", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_ring_trace_matches_oracle(oracle, cfg_idx, mode):
    cfg = ii.CONFIGS[cfg_idx]
    _drive(oracle, cfg.ring_N, cfg.ring_K, mode, seed=123 + cfg_idx,
           field_arrays_fn=lambda i: _fields(cfg_idx, 500 + i)[1], steps=200, gather=(mode == 0))


def test_ring_config2_shapes_and_host_push(oracle):
    cfg = ii.CONFIGS[2]
    base = _fields(2, 2)[1]

    def arrays(i):
        out = [a.copy() for a in base]
        out[1][:] += np.float32(i)  # make every batch distinct without regenerating 9 MB of logits
        out[0][0, 0] = i % 18
        return out
    _drive(oracle, cfg.ring_N, cfg.ring_K, 0, seed=9, field_arrays_fn=arrays, steps=120)
    _drive(oracle, 3, 2, 0, seed=10, field_arrays_fn=arrays, steps=12, host_src=True, gather=True)


def test_odd_field_sizes_and_partial_push(oracle):
    import paper_1912_00167_b200 as ip
    rng = np.random.default_rng(0)
    fb = [1, 15, 16, 17, 4099, 65536 + 3]
    ring = ip.ImpactBuffer(3, 2, fb, seed=5)
    for it in range(3):
        arrays = [rng.integers(0, 256, n, dtype=np.uint8) for n in fb]
        src = [torch.from_numpy(a).cuda() for a in arrays]
        src_partial = list(src)
        src_partial[4] = None  # appended later, like the target network's output at k = 0
        slot = ring.push(src_partial)
        assert slot == it
        ring.append(slot, 4, src[4])
        torch.cuda.synchronize()
        for f, a in enumerate(arrays):
            got = ring.slot_view(slot, f, torch.uint8, (fb[f],)).cpu().numpy()
            np.testing.assert_array_equal(got, a)
    assert ring.push([torch.zeros(n, dtype=torch.uint8, device="cuda") for n in fb]) is None
    ring.close()


def test_export_import_preserves_the_trace(oracle):
    import paper_1912_00167_b200 as ip
    fb = [64, 256]
    a = ip.ImpactBuffer(8, 3, fb, seed=42)
    src = [torch.zeros(n, dtype=torch.uint8, device="cuda") for n in fb]
    for _ in range(6):
        a.push(src)
    for _ in range(7):
        a.sample()
    blob = a.export_state()
    b = ip.ImpactBuffer(8, 3, fb, seed=0)
    b.import_state(blob)
    trace_a = [a.sample() for _ in range(5)] + [a.push(src)] + [a.sample() for _ in range(20)]
    trace_b = [b.sample() for _ in range(5)] + [b.push(src)] + [b.sample() for _ in range(20)]
    assert trace_a == trace_b and None in trace_a
    with pytest.raises(ip.ImpactError):
        ip.ImpactBuffer(4, 3, fb).import_state(blob)
    with pytest.raises(ip.ImpactError):
        b.import_state(blob[:-4])
    a.close(); b.close()


def test_library_owned_storage(oracle):
    import paper_1912_00167_b200 as ip
    fb = [1024]
    ring = ip.ImpactBuffer(2, 1, fb, library_owned_storage=True)
    x = torch.arange(1024, device="cuda").to(torch.uint8)
    dst = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    assert ring.push([x]) == 0
    assert ring.sample(gather_dst=[dst]) == (0, 0)
    torch.cuda.synchronize()
    assert torch.equal(dst, x)
    assert ring.sample() is None
    ring.close()


@pytest.mark.parametrize("row_shape,dtype", [((50, 18), torch.float32), ((7,), torch.float32), ((3,), torch.uint8),
                                             ((128, 18), torch.bfloat16), ((1,), torch.int32), ((5,), torch.float64)])
def test_gather_rows_is_bit_exact(row_shape, dtype):
    import paper_1912_00167_b200 as ip
    g = torch.Generator().manual_seed(1)
    n_src, n = 97, 1000
    src = torch.randint(0, 256, (n_src, *row_shape, torch.empty((), dtype=dtype).element_size()), dtype=torch.uint8,
                        generator=g).cuda()
    src = src.view(dtype).view(n_src, *row_shape)
    idx = torch.randint(0, n_src, (n,), generator=g).to(torch.int32).cuda()
    dst = torch.empty((n, *row_shape), dtype=dtype, device="cuda")
    ip.impact_gather_rows(src, idx, dst)
    torch.cuda.synchronize()
    want = src.view(torch.uint8).view(n_src, -1)[idx.long()]
    assert torch.equal(dst.view(torch.uint8).view(n, -1), want)


def test_gathered_trajectories_give_the_same_loss(oracle):
    """Index gather of trajectories feeds the loss kernel: compare with the oracle on the gathered batch."""
    import paper_1912_00167_b200 as ip
    import _parity as P
    cfg, b = ii.make_config(1)
    rng = np.random.default_rng(3)
    idx = rng.integers(0, cfg.B, size=20).astype(np.int32)
    gathered = {k: np.ascontiguousarray(v[idx]) for k, v in b.items()}
    dev = {}
    idx_d = torch.from_numpy(idx).cuda()
    for k, v in b.items():
        src = torch.from_numpy(v).cuda()
        dst = torch.empty((len(idx), *v.shape[1:]), dtype=src.dtype, device="cuda")
        ip.impact_gather_rows(src, idx_d, dst)
        dev[k] = dst
    torch.cuda.synchronize()
    for k in b:
        np.testing.assert_array_equal(dev[k].cpu().numpy(), gathered[k])
    P.check_categorical(oracle, {k: v.cpu().numpy() for k, v in dev.items()}, cfg.hyper)
