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


def _ring_with_candidates(cfg_idx, n_cand, N, K, mode, seed):
    """A ring plus `n_cand` candidate worker batches on the device and their address table for device_step."""
    import paper_1912_00167_b200 as ip
    names = ["actions", "rewards", "discounts", "worker_logp", "target_logits"]
    cands = []
    for i in range(n_cand):
        cfg, b = ii.make_config(cfg_idx, seed=700 + i)
        cands.append({k: torch.from_numpy(np.ascontiguousarray(v)).cuda() for k, v in b.items()})
    fb = [cands[0][n].numel() * cands[0][n].element_size() for n in names]
    ring = ip.ImpactBuffer(N, K, fb, seed=seed, sample_mode=mode)
    # per candidate: the four per-step fields (the slot's target-logits field is left for the first traversal), and
    # the candidate's fresh target logits as the pointer that is remembered with the slot
    table = torch.tensor([[c["actions"].data_ptr(), c["rewards"].data_ptr(), c["discounts"].data_ptr(),
                           c["worker_logp"].data_ptr(), 0, c["target_logits"].data_ptr()] for c in cands],
                         dtype=torch.int64, device="cuda")
    return cfg, ring, cands, table, names


@pytest.mark.parametrize("cfg_idx,mode,N,K", [(0, 0, 2, 2), (1, 0, 16, 2), (1, 1, 5, 3), (0, 0, 7, 1)])
def test_device_resident_bookkeeping_gives_the_oracles_trace(oracle, cfg_idx, mode, N, K):
    """The same script of pushes and draws, the bookkeeping on the device: every outcome (FULL, EMPTY, slot,
    traversal count) equals the oracle ring's, the slots hold the pushed bytes, the state survives the way back
    to the host, and a host-mode continuation agrees with the oracle as well."""
    import paper_1912_00167_b200 as ip
    seed = 90 + N
    cfg, ring, cands, table, names = _ring_with_candidates(cfg_idx, 3, N, K, mode, seed)
    ref = oracle.Ring(N, K, mode, seed=seed)
    record = ip.new_loss_inputs_record()
    fmap = {n: f for f, n in enumerate(names)}
    push_only = ring.prepare_device_step(push_sources=table)
    draw_only = ring.prepare_device_step(fmap, cands[0]["learner_logits"], cands[0]["values"],
                                         cands[0]["bootstrap_values"], record=record)
    both = ring.prepare_device_step(fmap, cands[0]["learner_logits"], cands[0]["values"], cands[0]["bootstrap_values"],
                                    push_sources=table, record=record)
    ring.device_begin()
    rng = np.random.default_rng(seed)
    want, where, pushes = [], {}, 0
    for step in range(120):
        u = rng.random()
        if u < 0.35:
            push_only()
            ops = ["push"]
        elif u < 0.75:
            draw_only()
            ops = ["draw"]
        else:
            both()
            ops = ["push", "draw"]
        for op in ops:
            if op == "push":
                st, slot = ref.push()
                want.append((1, -5 if st == ref.FULL else 0, -1 if st == ref.FULL else slot, 0))
                if st != ref.FULL:
                    where[slot] = pushes % 3
                    pushes += 1
            else:
                st, slot, k = ref.sample()
                want.append((2, -4, -1, 0) if st == ref.EMPTY else (2, 0, slot, k))
    got = ring.device_events()
    assert got == want
    assert ring.live() == ref.live()
    # the last successful draw's record names the slot's fields (and the fresh target logits at k = 0)
    last = [e for e in want if e[0] == 2 and e[1] == 0][-1]
    rec = ip.binding.impact_loss_inputs.from_buffer_copy(bytes(record.cpu().numpy())[:ip.binding.ctypes.sizeof(ip.binding.impact_loss_inputs)])
    assert (rec.status, rec.slot, rec.k_before) == (0, last[2], last[3])
    assert rec.actions == ring.slot_ptr(last[2], 0) and rec.worker_logp == ring.slot_ptr(last[2], 3)
    if last[3] == 0:
        assert rec.target_logits == cands[where[last[2]]]["target_logits"].data_ptr()
        assert rec.target_logits_copy == ring.slot_ptr(last[2], 4)
    else:
        assert rec.target_logits == ring.slot_ptr(last[2], 4) and not rec.target_logits_copy
    # payload: every live slot holds its candidate's bytes
    torch.cuda.synchronize()
    for slot, c in where.items():
        for f in range(4):
            view = ring.slot_view(slot, f, torch.uint8, (ring.field_bytes[f],))
            assert torch.equal(view, cands[c][names[f]].view(torch.uint8).reshape(-1))
    # back on the host the two rings keep agreeing
    ring.device_end()
    for _ in range(3 * N):
        got_h = ring.sample()
        st, slot, k = ref.sample()
        assert (got_h is None) == (st == ref.EMPTY)
        if got_h is not None:
            assert got_h == (slot, k)
    ring.close()


def test_learner_iterations_from_a_cuda_graph_with_device_bookkeeping(oracle):
    """Push-if-free, draw, loss with the inputs named by the draw's record: captured once into a CUDA graph and
    replayed.  Every iteration's loss terms equal those of the ordinary call on the batch the oracle ring says was
    drawn, and after a batch's first traversal its slot holds the target logits."""
    import paper_1912_00167_b200 as ip
    N, K, seed = 4, 2, 17
    cfg, ring, cands, table, names = _ring_with_candidates(1, 3, N, K, 0, seed)
    B, T, A = cfg.B, cfg.T, cfg.A
    ref = oracle.Ring(N, K, 0, seed=seed)
    learner = cands[0]  # the learner network's outputs: one fixed set of buffers
    coef = ip.Coefficients(clip_eps=0.3)
    ws = ip.new_workspace(B, T)
    record = ip.new_loss_inputs_record()
    out = dict(loss_terms=torch.zeros(8, device="cuda"), dlogits=torch.empty(B, T, A, device="cuda"),
               dvalues=torch.empty(B, T, device="cuda"))
    fmap = {n: f for f, n in enumerate(names)}
    step = ring.prepare_device_step(fmap, learner["learner_logits"], learner["values"], learner["bootstrap_values"],
                                    push_sources=table, record=record)
    loss = ip.prepare_loss_fwd_bwd_from_record(record, B, T, A, torch.float32, coef, workspace=ws, **out)
    ring.device_begin()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step.on_stream(side.cuda_stream)   # (warm-up outside the capture: first-use set-up of the kernels)
        loss.on_stream(side.cuda_stream)
    torch.cuda.synchronize()
    seen = [out["loss_terms"].clone()]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step.on_stream(side.cuda_stream)
            loss.on_stream(side.cuda_stream)
    for _ in range(11):
        graph.replay()
        torch.cuda.synchronize()
        seen.append(out["loss_terms"].clone())
    assert ip.impact_loss_workspace_status(ws) == 0
    # the oracle's trace for 12 iterations of push-then-draw, and the ordinary call on each drawn batch
    where, pushes = {}, 0
    want_out = dict(loss_terms=torch.zeros(8, device="cuda"), dlogits=torch.empty(B, T, A, device="cuda"),
                    dvalues=torch.empty(B, T, device="cuda"))
    for it in range(12):
        st, slot = ref.push()
        if st != ref.FULL:
            where[slot] = pushes % 3
            pushes += 1
        st, slot, k = ref.sample()
        assert st != ref.EMPTY
        c = cands[where[slot]]
        ip.impact_loss_fwd_bwd(learner["learner_logits"], c["target_logits"], c["worker_logp"], c["actions"],
                               c["rewards"], c["discounts"], learner["values"], learner["bootstrap_values"], coef,
                               workspace=ip.new_workspace(B, T), **want_out)
        torch.cuda.synchronize()
        assert torch.equal(seen[it], want_out["loss_terms"]), it
    events = ring.device_events()
    assert len(events) == 24 and all(e[1] in (0, -5) for e in events)
    # a slot whose current batch has been drawn holds that batch's target logits (appended by the loss call)
    drawn_since_push = {}
    for op, status, slot, k in events:
        if status != 0:
            continue
        drawn_since_push[slot] = (op == 2) if op == 2 else False
    for slot, was_drawn in drawn_since_push.items():
        if was_drawn:
            view = ring.slot_view(slot, 4, torch.float32, (B, T, A))
            assert torch.equal(view, cands[where[slot]]["target_logits"])
    ring.device_end()
    ring.close()
