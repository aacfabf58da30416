"""CPU checker for the expert-offload bookkeeping.  TEST INFRASTRUCTURE ONLY.

Pure integer simulation; shares no code with the CUDA/host library.

eq8_policy     -- the offloading rule exactly as the paper states it (Eq. 8,
                  Section 3.4.2): device memory holds the selected experts only.
lru_cache_sim  -- the same rule generalised to C >= k resident slots per layer
                  with least-recently-used eviction; with C = k it must move the
                  same experts as Eq. 8 (tested).

Pinned by tests: eq8_policy (hand-worked traces, the paper's capacity invariant),
lru_cache_sim (reduces to eq8_policy at C = k; invariants; hand-worked trace).
"""
from __future__ import annotations


def eq8_policy(trace):
    """trace: sequence of selected-expert lists, one per output token.
    Per token: if S != S_prev (as sets): every non-selected expert goes to the host,
    every selected expert to the device, S_prev <- S.  Returns, per token, the sorted
    list of experts that had to be brought to the device (those of S not already
    there), starting from an empty device."""
    on_device: set[int] = set()
    s_prev: set[int] | None = None
    fetched = []
    for sel in trace:
        S = set(int(e) for e in sel)
        moved = []
        if s_prev is None or S != s_prev:
            moved = sorted(S - on_device)
            on_device = set(S)          # N = E \ S leaves the device
            s_prev = S
        assert len(on_device) <= len(S)  # never more experts resident than active
        fetched.append(moved)
    return fetched


def lru_cache_sim(trace, n_experts: int, capacity: int, slot_bytes: int, initial=None):
    """Resident set of `capacity` slots.  Initially slot i holds expert initial[i]
    (default: expert i), slot 0 least recently used.  Per step, for each selected
    expert in the order given: resident -> mark most recently used; otherwise evict
    the least recently used resident expert that is not selected in this step, put the
    new expert in its slot and count slot_bytes of host->device traffic.
    Returns dict(fetches=[[(expert, slot), ...] per step], slots=[[expert per slot] per step],
    n_fetch, bytes, hits)."""
    if initial is None:
        initial = list(range(capacity))
    assert len(initial) == capacity and capacity <= n_experts
    slot_of = {int(e): s for s, e in enumerate(initial)}   # expert -> slot
    recency = [int(e) for e in initial]                    # least recent first
    fetches, slots_hist = [], []
    n_fetch = hits = 0
    for sel in trace:
        sel = [int(e) for e in sel]
        assert len(set(sel)) == len(sel) <= capacity
        step = []
        for e in sel:
            if e in slot_of:
                hits += 1
                recency.remove(e)
                recency.append(e)
                continue
            victim = next(v for v in recency if v not in sel)
            slot = slot_of.pop(victim)
            recency.remove(victim)
            slot_of[e] = slot
            recency.append(e)
            step.append((e, slot))
            n_fetch += 1
        assert len(slot_of) == capacity
        fetches.append(step)
        cur = [0] * capacity
        for e, s in slot_of.items():
            cur[s] = e
        slots_hist.append(cur)
    return {"fetches": fetches, "slots": slots_hist, "n_fetch": n_fetch,
            "bytes": n_fetch * slot_bytes, "hits": hits}
