"""The slot-and-flag protocol of the row-sharded fit, replayed on the CPU under random schedules.

Every rank repeats: write its vector into slot [step parity][rank] of every rank's buffer, publish the step in flag
[rank] of every buffer, wait until all flags of its OWN buffer show the step, read the `world` vectors of that slot.
The claim the kernel relies on: with only two slots, no rank ever reads a vector of another step than its own -- a
rank cannot be more than one step ahead of the slowest one, because it needs that rank's flag to go on.  Here the ranks
are small state machines advanced one action at a time in random order (publishing a flag after the stores is the only
ordering assumed, as on the device); every read is checked.  The buffer layout comes from the library.
"""
import random

import numpy as np

from paper_2308_10037_b200 import api


def run_schedule(world, n, steps, seed):
    rng = random.Random(seed)
    bytes_per_buffer = api.exchange_bytes(world, n)
    vec = ((n + 2) * 8 + 127) // 128 * 128
    assert bytes_per_buffer == 128 * world + 2 * world * vec          # flags, then [parity][rank] vectors
    flags = np.zeros((world, world), dtype=np.int64)                  # flags[owner][source]
    slots = np.zeros((world, 2, world), dtype=np.int64)               # slots[owner][parity][source] holds (step, source) coded
    # per rank: (step it works on, phase, next peer to store to / publish to)
    state = [dict(step=1, phase="store", k=0) for _ in range(world)]
    done = [False] * world
    reads = 0
    while not all(done):
        r = rng.randrange(world)
        s = state[r]
        if done[r]:
            continue
        if s["phase"] == "store":                                      # one store at a time, in any interleaving
            slots[s["k"], s["step"] & 1, r] = s["step"] * 1000 + r
            s["k"] += 1
            if s["k"] == world:
                s["phase"], s["k"] = "publish", 0
        elif s["phase"] == "publish":
            flags[s["k"], r] = s["step"]
            s["k"] += 1
            if s["k"] == world:
                s["phase"] = "wait"
        elif s["phase"] == "wait":
            if (flags[r] >= s["step"]).all():
                s["phase"] = "read"
        else:                                                          # read all vectors of the step from the own buffer
            for src in range(world):
                assert slots[r, s["step"] & 1, src] == s["step"] * 1000 + src, (r, s["step"], src)
                reads += 1
            s["step"] += 1
            s["phase"], s["k"] = "store", 0
            if s["step"] > steps:
                done[r] = True
    return reads


def test_two_slots_are_enough_under_any_schedule():
    for world in (1, 2, 3, 5):
        for seed in range(40):
            assert run_schedule(world, 28, steps=12, seed=seed) == world * world * 12


def test_one_slot_would_not_be():
    # the same replay with a single slot (parity ignored) must trip the check for some schedule: the test has teeth
    def run_one_slot(world, steps, seed):
        rng = random.Random(seed)
        flags = np.zeros((world, world), dtype=np.int64)
        slots = np.zeros((world, world), dtype=np.int64)
        state = [dict(step=1, phase="store", k=0) for _ in range(world)]
        done = [False] * world
        while not all(done):
            r = rng.randrange(world)
            s = state[r]
            if done[r]:
                continue
            if s["phase"] == "store":
                slots[s["k"], r] = s["step"] * 1000 + r
                s["k"] += 1
                if s["k"] == world:
                    s["phase"], s["k"] = "publish", 0
            elif s["phase"] == "publish":
                flags[s["k"], r] = s["step"]
                s["k"] += 1
                if s["k"] == world:
                    s["phase"] = "wait"
            elif s["phase"] == "wait":
                if (flags[r] >= s["step"]).all():
                    s["phase"] = "read"
            else:
                for src in range(world):
                    if slots[r, src] != s["step"] * 1000 + src:
                        return False
                s["step"] += 1
                s["phase"], s["k"] = "store", 0
                if s["step"] > steps:
                    done[r] = True
        return True
    assert not all(run_one_slot(3, 12, seed) for seed in range(40))
