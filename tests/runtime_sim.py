"""A small serving-loop simulation used by the runtime tests: host-side state of token tables
with per-request capacity, block lists and a free list, plus a dictionary "cache" that only
knows which (request, token id) pairs are alive.  Steps (append, evict, repack) can be run on
the oracle here and are replayed on the GPU by the GPU tests."""
import dataclasses

import numpy as np

from oracle import vto


class DictCache:
    """Ground truth of a token-evicting cache: a set of live token ids per request."""

    def __init__(self):
        self.live = {}

    def add(self, r, t):
        self.live.setdefault(r, set()).add(t)

    def remove(self, r, t):
        self.live.get(r, set()).discard(t)

    def live_tokens(self, r):
        return sorted(self.live.get(r, ()))


@dataclasses.dataclass
class ServingState:
    S: int
    num_blocks: int
    tt_offsets: np.ndarray      # int32 [R+1], capacity ranges
    tt_slots: np.ndarray        # int32 [sum capacity]
    keep: np.ndarray            # uint8
    tt_len: np.ndarray          # int32 [R]
    phys_len: np.ndarray        # int32 [R]
    block_lists: list           # per request int32 arrays
    free: list                  # free block ids, allocation order
    counters: dict = None       # optional: {"n_b": int32 [num_blocks], "live": int64 [1]} kept current by the steps

    def enable_counters(self):
        self.counters = dict(n_b=np.zeros(self.num_blocks, np.int32), live=np.zeros(1, np.int64))

    def recount(self):
        """After a structural change: the counters are recomputed from the tables."""
        n_b, _, live, _ = vto.block_liveness(self.S, self.num_blocks, self.bt_offsets, self.bt_blocks,
                                             self.tt_offsets, self.tt_slots, self.keep)
        self.counters["n_b"][:] = n_b
        self.counters["live"][0] = live

    @classmethod
    def empty(cls, S, capacities, block_lists, num_blocks=None, free=None):
        off = np.concatenate([[0], np.cumsum(capacities)]).astype(np.int32)
        R = len(capacities)
        nb = num_blocks if num_blocks is not None else int(max([b.max() for b in block_lists if len(b)] + [0])) + 1
        return cls(S, nb, off, np.full(off[-1], -1, np.int32), np.zeros(off[-1], np.uint8),
                   np.zeros(R, np.int32), np.zeros(R, np.int32),
                   [np.asarray(b, np.int32) for b in block_lists], list(free or []))

    @classmethod
    def random(cls, rng, S, R, capacity, num_blocks):
        free = rng.permutation(num_blocks).tolist()
        return cls.empty(S, [capacity] * R, [np.zeros(0, np.int32) for _ in range(R)], num_blocks, free)

    def set_block_lists(self, lists):
        self.block_lists = [np.asarray(b, np.int32) for b in lists]

    @property
    def R(self):
        return len(self.tt_len)

    @property
    def bt_offsets(self):
        return np.concatenate([[0], np.cumsum([len(b) for b in self.block_lists])]).astype(np.int32)

    @property
    def bt_blocks(self):
        return np.concatenate(self.block_lists + [np.zeros(0, np.int32)]).astype(np.int32)

    def grow_block_lists(self, new_len):
        """The scheduler's part of an append: hand out blocks so the new tokens have room."""
        for r in range(self.R):
            extra = max(0, int(new_len[r]) - int(self.tt_len[r]))
            need_blocks = -(-(int(self.phys_len[r]) + extra) // self.S)
            while len(self.block_lists[r]) < need_blocks and self.free:
                self.block_lists[r] = np.append(self.block_lists[r], np.int32(self.free.pop(0)))


@dataclasses.dataclass
class Append:
    new_len: np.ndarray

    def run_on_oracle(self, st, pool, truth):
        old = st.tt_len.copy()
        st.grow_block_lists(self.new_len)
        if st.counters is None:
            vto.sync_new_tokens(st.S, st.tt_offsets, st.tt_slots, st.keep, st.tt_len, st.phys_len, st.bt_offsets,
                                st.bt_blocks, self.new_len)
        else:
            vto.sync_new_tokens_counted(st.S, st.tt_offsets, st.tt_slots, st.keep, st.tt_len, st.phys_len,
                                        st.bt_offsets, st.bt_blocks, self.new_len, st.counters["n_b"],
                                        st.counters["live"])
        for r in range(st.R):
            for t in range(int(old[r]), int(st.tt_len[r])):
                if pool is not None:
                    pool[st.tt_slots[st.tt_offsets[r] + t]] = (r, t)      # the model writes the new token's K/V
                if truth is not None:
                    truth.add(r, t)


@dataclasses.dataclass
class Evict:
    victim_req: np.ndarray
    victim_tok: np.ndarray

    def run_on_oracle(self, st, pool, truth):
        if st.counters is None:
            vto.evict_tokens(st.tt_offsets, st.tt_len, st.keep, self.victim_req, self.victim_tok)
        else:
            vto.evict_tokens_counted(st.S, st.tt_offsets, st.tt_len, st.tt_slots, st.keep, self.victim_req,
                                     self.victim_tok, st.counters["n_b"], st.counters["live"])
        if truth is not None:
            for r, t in zip(self.victim_req.tolist(), self.victim_tok.tolist()):
                if 0 <= r < st.R and 0 <= t < st.tt_len[r]:
                    truth.remove(r, t)


@dataclasses.dataclass
class Repack:
    thr: tuple = (0, 0)
    num_free_limit: int = -1      # >= 0: pretend the free list is this short
    last_plan: object = None
    partial: dict = None          # options of the partial planner; None = whole-request plan
    waves: int = 0                # > 0: repack in this many waves (reclaimed blocks feed the next wave)

    def run_on_oracle(self, st, pool, truth):
        free = np.asarray(st.free, np.int32)
        nf = len(free) if self.num_free_limit < 0 else min(len(free), self.num_free_limit)
        if self.waves:
            p = vto.plan_waves(st.S, st.num_blocks, st.bt_offsets, st.bt_blocks, st.tt_offsets, st.tt_slots, st.keep,
                               free[:nf], self.waves, thr_num=self.thr[0], thr_den=self.thr[1], partial=self.partial)
            self.last_plan = p
            if pool is not None:
                vto.apply_moves_slab(pool, p.move_src, p.move_dst)        # list order = wave order
            vto.apply_moves(st.tt_offsets, st.tt_slots, st.keep, st.phys_len, p.new_tt_slots, p.req_status, S=st.S,
                            append_pos=p.req_append_pos)
            st.set_block_lists([p.new_bt_blocks[p.new_bt_offsets[r]:p.new_bt_offsets[r + 1]] for r in range(st.R)])
            st.free = p.free_out.tolist() + free[nf:].tolist()
            if st.counters is not None:
                st.recount()
            return
        if self.partial is None:
            p = vto.plan(st.S, st.bt_offsets, st.bt_blocks, st.tt_offsets, st.tt_slots, st.keep, free,
                         thr_num=self.thr[0], thr_den=self.thr[1], num_free=nf)
        else:
            p = vto.plan_partial(st.S, st.num_blocks, st.bt_offsets, st.bt_blocks, st.tt_offsets, st.tt_slots,
                                 st.keep, free, thr_num=self.thr[0], thr_den=self.thr[1], num_free=nf,
                                 **self.partial)
        self.last_plan = p
        if pool is not None:
            vto.apply_moves_slab(pool, p.move_src, p.move_dst)
        vto.apply_moves(st.tt_offsets, st.tt_slots, st.keep, st.phys_len, p.new_tt_slots, p.req_status, S=st.S,
                        new_bt_offsets=p.new_bt_offsets)
        st.set_block_lists([p.new_bt_blocks[p.new_bt_offsets[r]:p.new_bt_offsets[r + 1]] for r in range(st.R)])
        st.free = free[p.num_free_consumed:].tolist() + p.freed_blocks.tolist()
        if st.counters is not None:
            st.recount()


def random_serving_steps(rng, st, steps, partial_options=(), wave_options=()):
    """A seeded sequence of appends, evictions and repacks sized for ``st``.  ``partial_options``:
    option dicts of the partial planner to draw repacks from (empty: whole-request plans only);
    ``wave_options``: wave counts to draw from (0 = a single plan; empty: single plans only)."""
    R = st.R
    cap = np.diff(st.tt_offsets)
    length = np.zeros(R, np.int64)
    for i in range(steps):
        kind = i % 3
        if kind == 0:
            grow = rng.integers(0, 12, size=R)
            grow[rng.random(R) < 0.2] = 0
            length = np.minimum(length + grow, cap - 1)
            yield Append(length.astype(np.int32))
        elif kind == 1:
            n = int(rng.integers(1, 30))
            vr = rng.integers(0, R, size=n).astype(np.int32)
            vt = np.array([rng.integers(0, max(1, length[r])) for r in vr], np.int32)
            yield Evict(vr, vt)
        else:
            thr = [(0, 0), (1, 2), (3, 4)][int(rng.integers(0, 3))]
            limit = -1 if rng.random() < 0.7 else int(rng.integers(0, 6))
            partial = None
            if len(partial_options):
                partial = partial_options[int(rng.integers(0, len(partial_options)))]
            waves = 0
            if len(wave_options):
                waves = int(wave_options[int(rng.integers(0, len(wave_options)))])
                if waves and limit < 0:
                    limit = int(rng.integers(2, 12))          # waves are for short pools
            yield Repack(thr, limit, partial=partial, waves=waves)
