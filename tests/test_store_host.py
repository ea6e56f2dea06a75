"""The expert store's host logic without a GPU: allocator, event ordering and table updates run
against a fake copy engine that completes operations late and in adversarial order (tests/_fake_engine.py).
Checked: every "kernel" finds exactly the records it was promised, whatever the schedule; slot
maps equal the oracle allocator's; only misses are copied; canary words around the slot pool stay
intact; a protocol that leaves out a wait is caught by the same harness; and the hot path's
bookkeeping (hits, misses served on demand, deferred admissions) equals the oracle's."""
import ctypes as C

import numpy as np
import pytest

from oracle import moe_oracle as orc

from _fake_engine import FakeEngine

COPY, COMPUTE = 1, 2          # stream ids the fake engine is given
CANARY = 0xC3


@pytest.fixture(scope="module")
def lib():
    from paper_2609_18063_b200 import build
    build.build()
    import paper_2609_18063_b200 as m
    return m


class Rig:
    """A store of `n_layers` small layers on host memory, with canaries around pool and tables."""

    def __init__(self, lib, seed, S=4, E=16, K=2, n_layers=2):
        self.lib, self.S, self.E, self.K, self.L = lib, S, E, K, n_layers
        self.d = lib.make_desc(H=128, I=128, E=E, K=K, group=32, rank=0, n_adapters=1, n_slots=S, lora_scale=1.0)
        self.R = R = lib.record_bytes(self.d)
        rng = np.random.default_rng(seed)
        self.host = [np.ascontiguousarray(rng.integers(0, 256, (E, R), dtype=np.uint8)) for _ in range(n_layers)]
        pad = 4096
        self.raw = np.full(pad + n_layers * S * R + pad, CANARY, dtype=np.uint8)
        base = self.raw.ctypes.data
        off = (-base) % 256 + 256
        self.pool_off = off
        self.pool = self.raw[off:off + n_layers * S * R].reshape(n_layers, S, R)
        self.pool[:] = 0
        self.traw = np.full(64 + n_layers * E + 64, -0x3C3C3C3D, dtype=np.int32)
        toff = ((-self.traw.ctypes.data) % 16) // 4 + 16
        self.tables = self.traw[toff:toff + n_layers * E].reshape(n_layers, E)
        self.toff = toff
        self.eng = FakeEngine(seed)
        self.cengine = lib.make_copy_engine(self.eng)
        self.store = lib.Store(self.d, self.host, self.pool, self.tables, None, COPY, engine=self.cengine)
        self.violations = []

    def canaries_ok(self):
        n = self.L * self.S * self.R
        ok = (self.raw[:self.pool_off] == CANARY).all() and (self.raw[self.pool_off + n:] == CANARY).all()
        m = self.L * self.E
        return bool(ok and (self.traw[:self.toff] == -0x3C3C3C3D).all() and (self.traw[self.toff + m:] == -0x3C3C3C3D).all())

    def kernel(self, layer, P, expect_slots=None):
        """What the layer kernel would do when it runs: map P through the device table, read the slots."""
        def run():
            for i, e in enumerate(P):
                sl = int(self.tables[layer, e])
                if expect_slots is not None and expect_slots[i] < 0:
                    continue                              # a hot-path miss: served from the host tier
                if sl < 0 or sl >= self.S:
                    self.violations.append(("not resident", layer, e, sl))
                elif expect_slots is not None and sl != expect_slots[i]:
                    self.violations.append(("other slot", layer, e, sl, expect_slots[i]))
                elif not np.array_equal(self.pool[layer, sl], self.host[layer][e]):
                    self.violations.append(("wrong bytes", layer, e, sl))
        self.eng.kernel(COMPUTE, run)

    def step(self, layer, P, wait=True):
        slots, n_miss = self.lib.stage_experts_to_slots(self.store, layer, np.asarray(P, dtype=np.int32))
        if wait:
            self.store.wait_staged(layer, COMPUTE)
        self.kernel(layer, P)
        self.store.mark_computed(layer, COMPUTE)
        return slots.tolist(), n_miss


@pytest.mark.parametrize("seed", range(12))
def test_staged_path_under_adversarial_completion_order(lib, seed):
    rig = Rig(lib, seed)
    rng = np.random.default_rng(100 + seed)
    allocs = [orc.SlotAllocator(rig.E, rig.S) for _ in range(rig.L)]
    want_misses = 0
    for t in range(120):
        layer = int(rng.integers(rig.L))
        P = sorted(rng.choice(rig.E, rig.K, replace=False).tolist())
        slots, n_miss = rig.step(layer, P)
        want_slots, copies = allocs[layer].stage(P)
        assert slots == want_slots and n_miss == len(copies)
        want_misses += len(copies)
        rig.eng.run_some(int(rng.integers(0, 6)))         # the machine falls behind by a random amount
    assert rig.eng.drain()
    assert rig.violations == []
    assert rig.canaries_ok()
    for layer in range(rig.L):
        eos, soe = rig.store.snapshot(layer)
        assert eos.tolist() == allocs[layer].expert_of_slot and soe.tolist() == allocs[layer].slot_of_expert
        assert rig.tables[layer].tolist() == soe.tolist()
        for sl, e in enumerate(eos.tolist()):
            if e >= 0:
                assert np.array_equal(rig.pool[layer, sl], rig.host[layer][e])
    st = rig.store.stats()
    assert st["misses"] == want_misses and st["bytes_copied"] == want_misses * rig.R
    # record copies executed = misses; the rest of the engine's copies are table rows
    assert rig.eng.copies_done == want_misses + st["table_updates"]
    rig.store.close()


def test_the_harness_catches_a_protocol_that_skips_the_wait(lib):
    """Same traffic, but the compute side does not wait for the layer's staging copies: some schedule
    must show a kernel reading a slot before its record has landed.  (This is what the fake engine is for.)"""
    caught = 0
    for seed in range(8):
        rig = Rig(lib, seed)
        rng = np.random.default_rng(seed)
        for t in range(60):
            P = sorted(rng.choice(rig.E, rig.K, replace=False).tolist())
            rig.step(0, P, wait=False)
            rig.eng.run_some(int(rng.integers(0, 4)))
        rig.eng.drain()
        caught += 1 if rig.violations else 0
        rig.store.close()
    assert caught >= 6


def test_hits_enqueue_nothing_and_errors_leave_the_state_alone(lib):
    rig = Rig(lib, 3)
    rig.step(0, [1, 2])
    rig.eng.drain()
    n_ops = len(rig.eng.log)
    slots, n_miss = rig.lib.stage_experts_to_slots(rig.store, 0, np.array([1, 2], dtype=np.int32))
    assert n_miss == 0 and rig.eng.drain() and len(rig.eng.log) == n_ops          # sticky: nothing copied, nothing queued
    before = rig.store.snapshot(0)
    for bad, code in (([1, 1], -4), ([0, 99], -4), (list(range(rig.S + 1)), -3)):
        with pytest.raises(lib.EdgError) as ei:
            rig.lib.stage_experts_to_slots(rig.store, 0, np.array(bad, dtype=np.int32))
        assert ei.value.code == code
    after = rig.store.snapshot(0)
    assert before[0].tolist() == after[0].tolist() and before[1].tolist() == after[1].tolist()
    rig.store.close()


@pytest.mark.parametrize("seed,admit_after", [(0, 1), (1, 1), (2, 2), (3, 3)])
def test_hot_path_bookkeeping_matches_the_oracle(lib, seed, admit_after):
    """The hot executor path on the host: S - K hot slots, the last K transient.  A step sees the table
    as it was; its misses are served on demand; admissions are queued behind the step's compute."""
    S, K, E = 7, 2, 16
    rig = Rig(lib, seed, S=S, E=E, K=K, n_layers=1)
    rig.store.set_hot(True, admit_after)
    hot = orc.HotSetAllocator(E, S - K, admit_after)
    rng = np.random.default_rng(50 + seed)
    pop = np.array([6.0] * 4 + [1.0] * (E - 4)); pop /= pop.sum()        # a few popular experts
    for t in range(200):
        P = sorted(rng.choice(E, K, replace=False, p=pop).tolist())
        slots, n_miss = rig.lib.stage_experts_to_slots(rig.store, 0, np.asarray(P, dtype=np.int32))
        want, adm = hot.step(P)
        assert slots.tolist() == want and n_miss == sum(1 for s in want if s < 0)
        rig.store.wait_staged(0, COMPUTE)
        rig.kernel(0, P, expect_slots=want)
        rig.store.mark_computed(0, COMPUTE)               # the admissions of this step go out here
        rig.eng.run_some(int(rng.integers(0, 8)))
    assert rig.eng.drain() and rig.violations == [] and rig.canaries_ok()
    eos, soe = rig.store.snapshot(0)
    assert eos.tolist()[:S - K] == hot.expert_of_slot and eos.tolist()[S - K:] == [-1] * K
    assert soe.tolist() == hot.slot_of_expert
    hs = rig.store.hot_stats()
    assert (hs["hits"], hs["misses"], hs["admitted"]) == (hot.hits, hot.misses, hot.admitted)
    assert hs["bytes_direct"] == hot.misses * rig.R and rig.store.stats()["bytes_copied"] == hot.admitted * rig.R
    assert hs["hits"] > hs["misses"] * 0.3               # the popular experts do get cached
    for sl, e in enumerate(hot.expert_of_slot):
        if e >= 0:
            assert np.array_equal(rig.pool[0, sl], rig.host[0][e])
    rig.store.close()


def test_hot_path_needs_room_and_an_early_switch(lib):
    rig = Rig(lib, 0, S=2, K=2)
    with pytest.raises(lib.EdgError) as ei:
        rig.store.set_hot(True, 1)
    assert ei.value.code == -3                               # no slot left for a hot set
    rig.store.close()
    rig = Rig(lib, 0, S=6, K=2)
    rig.step(0, [1, 2])
    with pytest.raises(lib.EdgError):
        rig.store.set_hot(True, 1)                           # after the first staging call
    rig.store.close()


@pytest.mark.parametrize("seed", range(4))
def test_whole_layer_loads_as_a_double_buffer(lib, seed):
    """The whole-layer path on the host: a store of two pool layers serves a deeper model.  Layer l+1 is
    loaded into the other pool layer while the "kernel" of layer l runs; each kernel must find all E
    records of ITS model layer, whatever the schedule, and a pool layer is only overwritten behind the
    compute that last read it."""
    E = 8
    rig = Rig(lib, seed, S=E, E=E, K=2, n_layers=2)
    rng = np.random.default_rng(seed)
    depth = 7
    model = [np.ascontiguousarray(rng.integers(0, 256, (E, rig.R), dtype=np.uint8)) for _ in range(depth)]

    def kernel(pool_layer, l):
        def run():
            if rig.tables[pool_layer].tolist() != list(range(E)):
                rig.violations.append(("table", l))
            elif not np.array_equal(rig.pool[pool_layer], model[l]):
                rig.violations.append(("bytes", l))
        rig.eng.kernel(COMPUTE, run)

    rig.store.load_whole_layer(0, model[0])
    for l in range(depth):
        if l + 1 < depth:
            rig.store.load_whole_layer((l + 1) % 2, model[l + 1])     # runs while layer l computes
        rig.store.wait_staged(l % 2, COMPUTE)
        kernel(l % 2, l)
        rig.store.mark_computed(l % 2, COMPUTE)
        rig.eng.run_some(int(rng.integers(0, 5)))
    assert rig.eng.drain() and rig.violations == [] and rig.canaries_ok()
    assert rig.store.stats()["bytes_copied"] == depth * E * rig.R
    eos, soe = rig.store.snapshot(1)
    assert eos.tolist() == list(range(E)) and soe.tolist() == list(range(E))
    # a pool smaller than the layer cannot take a whole layer
    small = Rig(lib, seed, S=4, E=E, K=2, n_layers=1)
    with pytest.raises(lib.EdgError) as ei:
        small.store.load_whole_layer(0)
    assert ei.value.code == -3
    small.store.close()
    rig.store.close()
