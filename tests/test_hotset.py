"""Hot-set slot table (Definition 5.1): host bookkeeping against a fake maintenance stream on the CPU, and the whole
path through the slot table on the GPU against the oracle applied to the resolved adapters."""
import ctypes

import numpy as np
import pytest

import paper_2603_15965_b200 as M
from paper_2603_15965_b200 import binding as B


class FakeStream:
    """Copies and events are queued and only take effect on flush(): what a stream does, without a GPU.  Destinations are
    plain host buffers standing in for device memory."""

    def __init__(self):
        self.queue, self.log, self.events, self.next_event = [], [], {}, 1
        self.backend = B._HotsetBackendC(B.COPY_FN(self._copy), B.EVENT_RECORD_FN(self._record), B.EVENT_DONE_FN(self._done),
                                         B.EVENT_DESTROY_FN(self._destroy), None)

    def _copy(self, dst, src, nbytes, stream, user):
        data = ctypes.string_at(src, nbytes)              # the source may be reused by the caller: snapshot at enqueue
        self.queue.append(("copy", dst, data))
        return 0

    def _record(self, event_pp, stream, user):
        if not event_pp[0]:
            event_pp[0] = self.next_event
            self.next_event += 1
        self.events[event_pp[0]] = False
        self.queue.append(("event", event_pp[0], None))
        return 0

    def _done(self, event, user):
        return 1 if self.events.get(event, False) else 0

    def _destroy(self, event, user):
        pass

    def flush(self):
        for kind, a, b in self.queue:
            if kind == "copy":
                ctypes.memmove(a, b, len(b))
                self.log.append((a, len(b)))
            else:
                self.events[a] = True
        self.queue = []


def _make(S=3, M_=2, n_catalog=10, slot_bytes=64):
    fs = FakeStream()
    table = np.full(n_catalog, -1, np.int32)
    stack = np.zeros((S, slot_bytes), np.uint8)
    hs = M.HotSet(S, M_, n_catalog, table.ctypes.data, backend=fs.backend)
    return fs, table, stack, hs


class _Host:          # what HotSet.upload needs of a tensor
    def __init__(self, a):
        self.a = a

    def numel(self):
        return self.a.size

    def element_size(self):
        return self.a.itemsize

    def data_ptr(self):
        return self.a.ctypes.data


def _load(hs, fs, stack, adapter, flush=True):
    slot, fresh, evicted = hs.begin_load(adapter, stream=0)
    if fresh:
        w = np.full(stack.shape[1], adapter + 1, np.uint8)
        lib = M.load_library()
        assert lib.molora_hotset_upload(hs.h, slot, ctypes.c_void_p(stack.ctypes.data), ctypes.c_void_p(w.ctypes.data), w.size, None) == 0
        hs.commit(slot, stream=0)
    if flush:
        fs.flush()
    return slot, evicted


def test_slots_fill_in_order_and_become_resident_only_after_the_copies():
    fs, table, stack, hs = _make()
    slot, evicted = _load(hs, fs, stack, 7, flush=False)
    assert (slot, evicted) == (0, -1)
    assert hs.slot_of(7) == -1 and table[7] == -1                 # enqueued, not landed: neither host nor device see it
    with pytest.raises(M.MoloraError) as e:
        hs.pin(7)
    assert e.value.status == B.ERR_NOT_RESIDENT
    fs.flush()
    assert hs.slot_of(7) == 0 and table[7] == 0 and np.all(stack[0] == 8) and hs.adapter_in(0) == 7
    # the table entry is written AFTER the weights (stream order): last copy of the log is the 4-byte table update
    assert fs.log[-1] == (table.ctypes.data + 4 * 7, 4) and fs.log[-2][1] == stack.shape[1]
    assert _load(hs, fs, stack, 2)[0] == 1 and _load(hs, fs, stack, 9)[0] == 2
    assert _load(hs, fs, stack, 2) == (1, -1)                     # already resident: same slot, nothing evicted


def test_eviction_takes_the_least_recently_pinned_unpinned_slot_and_never_a_pinned_one():
    fs, table, stack, hs = _make()
    for a in (4, 5, 6):
        _load(hs, fs, stack, a)
    s4 = hs.pin(4); hs.unpin(s4)
    s5 = hs.pin(5)                                                # stays pinned: a step is in flight
    s6 = hs.pin(6); hs.unpin(s6)
    fs.log.clear()
    slot, evicted = _load(hs, fs, stack, 1, flush=False)
    assert (slot, evicted) == (s4, 4)                             # 4 was pinned longest ago; 5 is pinned
    assert hs.slot_of(4) == -1 and hs.slot_of(1) == -1            # evicted at once on the host, new one not yet there
    fs.flush()
    # device order: clear the old entry, then the weights, then the new entry
    assert [n for _, n in fs.log] == [4, stack.shape[1], 4] and fs.log[0][0] == table.ctypes.data + 4 * 4
    assert table[4] == -1 and table[1] == s4 and np.all(stack[s4] == 2)
    slot, evicted = _load(hs, fs, stack, 0)
    assert (slot, evicted) == (s6, 6)
    hs.pin(1); hs.pin(0)
    with pytest.raises(M.MoloraError) as e:                       # all three pinned: nothing may be evicted
        hs.begin_load(8, stream=0)
    assert e.value.status == B.ERR_BUSY
    hs.unpin(s5)
    assert hs.begin_load(8, stream=0) == (s5, True, 5)


def test_arguments_and_a_slot_being_filled_is_not_a_victim():
    fs, table, stack, hs = _make(S=2)
    lib = M.load_library()
    assert lib.molora_hotset_create(200, 2, 10, ctypes.c_void_p(table.ctypes.data), None, ctypes.byref(ctypes.c_void_p())) == 2
    assert lib.molora_hotset_create(2, 2, 10, None, None, ctypes.byref(ctypes.c_void_p())) == 1
    a, fresh, _ = hs.begin_load(3, stream=0)
    b, _, _ = hs.begin_load(4, stream=0)
    assert fresh and hs.begin_load(3, stream=0) == (a, False, -1)     # already on its way
    with pytest.raises(M.MoloraError) as e:                       # both slots are being filled
        hs.begin_load(5, stream=0)
    assert e.value.status == B.ERR_BUSY
    assert lib.molora_hotset_commit(hs.h, 7, None) == 1 and lib.molora_hotset_unpin(hs.h, a) == 1
    hs.commit(a, stream=0); hs.commit(b, stream=0); fs.flush()
    assert lib.molora_hotset_commit(hs.h, a, None) == 1           # not being loaded any more
    assert sorted([hs.slot_of(3), hs.slot_of(4)]) == [0, 1]


@pytest.mark.gpu
def test_route_group_apply_through_the_slot_table_matches_the_oracle_on_the_resolved_adapters():
    import torch
    import oracle
    from paper_2603_15965_b200 import workloads as W
    from _harness import assert_close, dev_tensor, to_f64

    S, Mm, n_catalog, d_in, d_out, rank, N = 3, 2, 6, 256, 192, 16, 900
    rng = np.random.default_rng(51)
    breaks = np.array([0, 500, 1000], np.int32)
    # catalog weights on the host (pinned), one (M, d_in, r) / (M, r, d_out) block per adapter
    cat_A = W.round_to_bf16((rng.standard_normal((n_catalog, Mm, d_in, rank)) * d_in ** -0.5).astype(np.float32))
    cat_B = W.round_to_bf16((rng.standard_normal((n_catalog, Mm, rank, d_out)) * 0.1).astype(np.float32))
    hA = torch.from_numpy(W.bf16_bits(cat_A)).view(torch.bfloat16).pin_memory()
    hB = torch.from_numpy(W.bf16_bits(cat_B)).view(torch.bfloat16).pin_memory()
    A_hot = torch.zeros(S, Mm, d_in, rank, dtype=torch.bfloat16, device="cuda")
    B_hot = torch.zeros(S, Mm, rank, d_out, dtype=torch.bfloat16, device="cuda")
    table = torch.full((n_catalog,), -1, dtype=torch.int32, device="cuda")
    hs = M.HotSet(S, Mm, n_catalog, table)
    side = torch.cuda.Stream()

    def load(adapter):
        slot, fresh, evicted = hs.begin_load(adapter, stream=side)
        if fresh:
            hs.upload(slot, A_hot, hA[adapter], stream=side)
            hs.upload(slot, B_hot, hB[adapter], stream=side)
            hs.commit(slot, stream=side)
        return slot, evicted

    def step(adapters_of_requests, x, y, ids, adapter_id):
        """route -> group -> apply with the adapters pinned for the duration of the step; returns (h, r)."""
        slots = [hs.pin(a) for a in sorted(set(adapters_of_requests))]
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        r = M.molora_route_hotset(dev_tensor(ids, "i"), dev_tensor(adapter_id, "i"), dev_tensor(breaks, "i"), table, S,
                                  dev_status=status)
        counts, offsets, perm = M.molora_group(r, S * Mm)
        yd = dev_tensor(y, "bf16")
        M.molora_apply(dev_tensor(x, "bf16"), yd, A_hot.view(S * Mm, d_in, rank), B_hot.view(S * Mm, rank, d_out), offsets, perm)
        torch.cuda.synchronize()
        for s in slots:
            hs.unpin(s)
        return yd, r.cpu().numpy(), int(status.item())

    for a in (4, 1, 5):
        load(a)
    side.synchronize()
    assert sorted(hs.slot_of(a) for a in (4, 1, 5)) == [0, 1, 2] and hs.slot_of(0) == -1

    def batch(seed, adapters):
        g = np.random.default_rng(seed)
        req = g.choice(adapters, size=N // 50)                         # 18 requests of 50 tokens, one adapter each
        adapter_id = np.repeat(req, 50).astype(np.int32)
        ids = g.integers(0, 1000, size=N).astype(np.int32)
        x = W.round_to_bf16(g.standard_normal((N, d_in), dtype=np.float32))
        y = W.round_to_bf16(g.standard_normal((N, d_out), dtype=np.float32))
        return req, adapter_id, ids, x, y

    def check(h, r, adapter_id, ids, x, y, resident):
        # oracle on the RESOLVED adapters: the catalog's weights indexed by adapter * M + modality, never by slot
        modality = oracle.route_vocab(ids, breaks)
        r_cat = np.where(np.isin(adapter_id, resident), adapter_id * Mm + modality, -1).astype(np.int32)
        ref, _ = oracle.apply(x, y, cat_A.reshape(n_catalog * Mm, d_in, rank), cat_B.reshape(n_catalog * Mm, rank, d_out), r_cat)
        assert_close(to_f64(h), ref, what="apply through the slot table")
        slot = np.array([hs.slot_of(int(a)) for a in adapter_id])
        assert np.array_equal(r, np.where(slot >= 0, slot * Mm + modality, -1))

    req, adapter_id, ids, x, y = batch(1, [4, 1, 5])
    h, r, status = step(req, x, y, ids, adapter_id)
    check(h, r, adapter_id, ids, x, y, [4, 1, 5])
    assert status == 0
    # tokens of an adapter that is not resident stay unrouted (h = y) and are flagged; nothing faults
    req, adapter_id, ids, x, y = batch(2, [4, 0])
    h, r, status = step([4], x, y, ids, adapter_id)
    check(h, r, adapter_id, ids, x, y, [4])
    assert status & 1
    # refill: adapter 0 takes the slot of the least recently pinned adapter (1 or 5, both unpinned; 4 was pinned last)
    hs.pin(4)
    slot, evicted = load(0)
    side.synchronize()
    assert evicted in (1, 5) and hs.slot_of(evicted) == -1 and hs.slot_of(0) == slot
    hs.unpin(hs.slot_of(4))
    resident = [a for a in (4, 1, 5, 0) if a != evicted]
    req, adapter_id, ids, x, y = batch(3, resident)
    h, r, status = step(req, x, y, ids, adapter_id)
    check(h, r, adapter_id, ids, x, y, resident)
    assert status == 0
    hs.close()
