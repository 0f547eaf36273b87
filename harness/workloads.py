"""Seeded synthetic inputs for the repack path: request lengths, eviction masks,
block and token tables, free lists and the deterministic K/V pool fill.

This module only *generates inputs*.  It contains none of the method's arithmetic
(no live counts, no destination assignment, no copies) so that the CPU oracle and the
CUDA library can both be fed from it while sharing nothing else.

The five generators follow the five workload shapes the build is measured on:

  1. ``tiny``        1 layer, 2 KV heads, head_dim 64, S=16, 4 requests of 100-300 tokens,
                     Random eviction with keep probability 0.5.
  2. ``llama8b_h2o`` 32 layers, 8 KV heads, head_dim 128, S=16, 64 requests of 1k-4k tokens,
                     H2O-style mask (4 sink + 64 recent + top-k by lognormal score, 20 % budget).
  3. ``mistral7b_random`` same shape, 256 requests of 512-2048 tokens, Random eviction with
                     a per-request keep ratio drawn from U(0.3, 0.7).
  4. ``longctx_scissor`` 28 layers, 4 KV heads, head_dim 128, S=32, 32 requests of 16k-32k
                     tokens, Scissorhands-style mask (256 recent + Binomial(n_obs, 0.2) >= 2).
  5. ``steady_state`` shape of 2 with S in {16, 32}, 512 requests of 256-8k tokens that have
                     already been evicted and packed once (token tables with -1 holes),
                     second H2O-style eviction pass, repack only requests whose live
                     fraction is below 1/2.

They stand in for the ShareGPT / LongBench request mixes the paper evaluates on
(Section 5 set-up): only lengths, tables, masks and bytes reach the repack path, so only
their shapes are reproduced.  Every draw comes from ``numpy.random.Generator(PCG64(seed))``
in a fixed order: lengths, per-request mask parameters, per-token draws (request-major),
then the physical block permutation.

Every generator takes ``scale`` knobs (requests, length range, layers) so that tests can
run the same recipe at sizes the CPU oracle finishes in seconds.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import numpy as np

# --------------------------------------------------------------------------------------
# K/V pool fill: a counter-based generator, identical on host (numpy, below) and device
# (the fill kernel of the harness library).  Only integer arithmetic, one exact
# int->float32 conversion, one float32 multiply and an integer round-to-bf16 are used, so
# the two implementations agree bit for bit.
#   counter = ((kv * L + layer) * slots_per_layer + slot) * row_elems + elem
#   h       = splitmix64(counter + seed * GOLDEN)
#   s       = sum of the four 16-bit fields of h          (Irwin-Hall, n = 4)
#   x       = float32(s - 131070) * FILL_SCALE             (mean 0, variance 1)
#   value   = bf16 round-to-nearest-even of x
# --------------------------------------------------------------------------------------
FILL_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
FILL_MEAN = 131070  # 4 * 65535 / 2
# 1 / sqrt(4 * (65536**2 - 1) / 12), rounded to float32 once and used as that float32.
FILL_SCALE = np.float32(1.0 / math.sqrt(4.0 * (65536.0 ** 2 - 1.0) / 12.0))


def _splitmix64(x: np.ndarray) -> np.ndarray:
    x = x.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        x += FILL_GOLDEN
        x ^= x >> np.uint64(30)
        x *= np.uint64(0xBF58476D1CE4E5B9)
        x ^= x >> np.uint64(27)
        x *= np.uint64(0x94D049BB133111EB)
        x ^= x >> np.uint64(31)
    return x


def fill_values(counter: np.ndarray, seed: int) -> np.ndarray:
    """bf16 bit patterns (uint16) of the pool fill at the given element counters."""
    with np.errstate(over="ignore"):
        h = _splitmix64(counter.astype(np.uint64) + np.uint64(seed) * FILL_GOLDEN)
    s = ((h & np.uint64(0xFFFF)) + ((h >> np.uint64(16)) & np.uint64(0xFFFF))
         + ((h >> np.uint64(32)) & np.uint64(0xFFFF)) + (h >> np.uint64(48))).astype(np.int64)
    x = (s - FILL_MEAN).astype(np.float32) * FILL_SCALE
    bits = x.view(np.uint32)
    rounded = (bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def fill_rows(seed: int, kv: int, layer: int, num_layers: int, slots_per_layer: int,
              row_elems: int, slots: np.ndarray) -> np.ndarray:
    """Pool pre-state of the given slots of one (K|V, layer) slab: uint16 [len(slots), row_elems]."""
    slots = np.asarray(slots, dtype=np.uint64)
    base = (np.uint64(kv * num_layers + layer) * np.uint64(slots_per_layer) + slots) * np.uint64(row_elems)
    counter = base[:, None] + np.arange(row_elems, dtype=np.uint64)[None, :]
    return fill_values(counter, seed)


def fill_slab(seed: int, kv: int, layer: int, num_layers: int, slots_per_layer: int,
              row_elems: int) -> np.ndarray:
    """Pool pre-state of one whole (K|V, layer) slab: uint16 [slots_per_layer, row_elems]."""
    return fill_rows(seed, kv, layer, num_layers, slots_per_layer, row_elems,
                     np.arange(slots_per_layer, dtype=np.uint64))


def fill_slab_address(kv: int, layer: int, slots_per_layer: int, row_elems: int) -> np.ndarray:
    """Address-encoding fill of one (K|V, layer) slab, uint16 [slots_per_layer, row_elems]: every 8 bytes
    of a row say where the row was filled -- low 32-bit word = slot, high word = pool (bit 31), layer
    (bits 16..30), index of the 8-byte group in the row (bits 0..15).  Identical to the harness kernel;
    a row found in the wrong place names the place it came from (``decode_row_address``)."""
    groups = row_elems // 4
    out = np.empty((slots_per_layer, groups, 2), dtype=np.uint32)
    out[:, :, 0] = np.arange(slots_per_layer, dtype=np.uint32)[:, None]
    out[:, :, 1] = (np.uint32(kv) << np.uint32(31)) | (np.uint32(layer) << np.uint32(16)) | np.arange(groups, dtype=np.uint32)[None, :]
    return out.reshape(slots_per_layer, groups * 2).view(np.uint16).reshape(slots_per_layer, row_elems)


def decode_row_address(row: np.ndarray):
    """(kv, layer, slot) an address-filled row says it came from, or None when its 8-byte groups disagree
    (bytes of several rows, or not an address fill at all)."""
    w = np.ascontiguousarray(row).view(np.uint32).reshape(-1, 2)
    slot, hi = w[:, 0], w[:, 1]
    kv, layer, group = hi >> np.uint32(31), (hi >> np.uint32(16)) & np.uint32(0x7FFF), hi & np.uint32(0xFFFF)
    ok = (slot == slot[0]).all() and (kv == kv[0]).all() and (layer == layer[0]).all() and \
        (group == np.arange(len(group), dtype=np.uint32)).all()
    return (int(kv[0]), int(layer[0]), int(slot[0])) if ok else None


# --------------------------------------------------------------------------------------
@dataclasses.dataclass
class Workload:
    """One repack problem: shape, CSR tables, masks, free list (all numpy, host)."""
    name: str
    num_layers: int
    num_kv_heads: int
    head_dim: int
    block_size: int
    num_blocks: int
    bt_offsets: np.ndarray      # int32 [R+1]
    bt_blocks: np.ndarray       # int32 [bt_offsets[R]]
    tt_offsets: np.ndarray      # int32 [R+1]
    tt_slots: np.ndarray        # int32 [T]  block*S+off, or -1
    keep: np.ndarray            # uint8 [T]
    free_blocks: np.ndarray     # int32 [num_free]
    select: Optional[np.ndarray] = None   # uint8 [R] or None
    thr_num: int = 0
    thr_den: int = 0            # 0 = no threshold
    seed: int = 0
    elem_bytes: int = 2
    notes: dict = dataclasses.field(default_factory=dict)

    @property
    def num_requests(self) -> int:
        return len(self.tt_offsets) - 1

    @property
    def num_tokens(self) -> int:
        return int(self.tt_offsets[-1])

    @property
    def row_elems(self) -> int:
        return self.num_kv_heads * self.head_dim

    @property
    def row_bytes(self) -> int:
        return self.row_elems * self.elem_bytes

    @property
    def token_bytes(self) -> int:
        """K and V bytes of one token over all layers (2 * L * H * D * dtype size)."""
        return kv_bytes_per_token(self.num_layers, self.num_kv_heads, self.head_dim, self.elem_bytes)

    @property
    def slots_per_layer(self) -> int:
        return self.num_blocks * self.block_size

    @property
    def slab_bytes(self) -> int:
        return self.slots_per_layer * self.row_bytes

    @property
    def pool_bytes(self) -> int:
        """Bytes of ONE pool (K or V) over all layers."""
        return self.num_layers * self.slab_bytes


def kv_bytes_per_token(num_layers: int, num_kv_heads: int, head_dim: int, elem_bytes: int) -> int:
    return 2 * num_layers * num_kv_heads * head_dim * elem_bytes


# --------------------------------------------------------------------------------------
# masks (inputs from an eviction policy; the path under test never looks inside them)
# --------------------------------------------------------------------------------------
def h2o_mask(ids: np.ndarray, length: int, score: np.ndarray, budget: int,
             sink: int = 4, recent: int = 64) -> np.ndarray:
    """H2O-style keep decision over the resident logical ids ``ids`` of a request of
    ``length`` tokens: the first ``sink`` ids, the last ``recent`` ids and the highest-score
    ids of the middle up to ``budget`` kept tokens in total (ties -> lower id)."""
    ids = np.asarray(ids, dtype=np.int64)
    is_sink = ids < sink
    is_recent = ids >= length - recent
    fixed = is_sink | is_recent
    k = max(0, budget - int(fixed.sum()))
    keep = fixed.copy()
    mid = np.flatnonzero(~fixed)
    if k > 0 and len(mid) > 0:
        order = np.argsort(-score[ids[mid]], kind="stable")
        keep[mid[order[:k]]] = True
    return keep


def _deal_blocks(rng: np.random.Generator, nb: np.ndarray, extra_free: int):
    """Physical ids: a seeded permutation of [0, NB) dealt to requests round-robin, one
    block per request per turn (interleaved on-demand allocation).  Returns
    (NB, bt_offsets, bt_blocks, free_blocks)."""
    R = len(nb)
    total = int(nb.sum())
    NB = total + extra_free
    perm = rng.permutation(NB).astype(np.int32)
    bt_offsets = np.zeros(R + 1, dtype=np.int32)
    np.cumsum(nb, out=bt_offsets[1:])
    bt_blocks = np.empty(total, dtype=np.int32)
    # turn j hands one block to every request with j < nb[r], in request order
    order_r = np.argsort(nb, kind="stable")
    nb_sorted = nb[order_r]
    cursor = 0
    maxnb = int(nb.max()) if R else 0
    for j in range(maxnb):
        first = int(np.searchsorted(nb_sorted, j, side="right"))
        rs = np.sort(order_r[first:])
        bt_blocks[bt_offsets[rs] + j] = perm[cursor:cursor + len(rs)]
        cursor += len(rs)
    free_blocks = np.sort(perm[cursor:]).astype(np.int32)
    return NB, bt_offsets, bt_blocks, free_blocks


def _assemble(name, shape, S, lens, resident_lists, keep_lists, rng, seed,
              select=None, thr=(0, 0), headroom=256, notes=None) -> Workload:
    """Common tail of every generator: block counts, permutation, tables, free list.
    ``resident_lists[r]`` = ascending logical ids that own a physical slot (None = all)."""
    L, H, D = shape
    R = len(lens)
    resident_n = np.array([lens[r] if resident_lists[r] is None else len(resident_lists[r])
                           for r in range(R)], dtype=np.int64)
    nb = (resident_n + S - 1) // S
    live_n = np.array([int(k.sum()) for k in keep_lists], dtype=np.int64)
    dst_n = (live_n + S - 1) // S
    if thr[1]:
        # size the free list for the requests the live-fraction threshold lets through
        dst_n = np.where(live_n * thr[1] < thr[0] * nb * S, dst_n, 0)
    dst_total = int(dst_n.sum())
    NB, bt_offsets, bt_blocks, free_blocks = _deal_blocks(rng, nb, dst_total + headroom)
    tt_offsets = np.zeros(R + 1, dtype=np.int32)
    np.cumsum(lens, out=tt_offsets[1:])
    T = int(tt_offsets[-1])
    tt_slots = np.full(T, -1, dtype=np.int32)
    keep = np.zeros(T, dtype=np.uint8)
    for r in range(R):
        ids = np.arange(lens[r]) if resident_lists[r] is None else np.asarray(resident_lists[r])
        pos = np.arange(len(ids))
        blocks = bt_blocks[bt_offsets[r]:bt_offsets[r + 1]]
        if len(ids):
            tt_slots[tt_offsets[r] + ids] = blocks[pos // S].astype(np.int64) * S + pos % S
        keep[tt_offsets[r]:tt_offsets[r + 1]] = keep_lists[r].astype(np.uint8)
    return Workload(name=name, num_layers=L, num_kv_heads=H, head_dim=D, block_size=S,
                    num_blocks=NB, bt_offsets=bt_offsets, bt_blocks=bt_blocks,
                    tt_offsets=tt_offsets, tt_slots=tt_slots, keep=keep,
                    free_blocks=free_blocks, select=select, thr_num=thr[0], thr_den=thr[1],
                    seed=seed, notes=notes or {})


# --------------------------------------------------------------------------------------
# the five workloads
# --------------------------------------------------------------------------------------
def tiny(seed: int = 0, requests: int = 4, lo: int = 100, hi: int = 300, p_keep: float = 0.5,
         layers: int = 1, heads: int = 2, head_dim: int = 64, block_size: int = 16) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    lens = rng.integers(lo, hi + 1, size=requests)
    keeps = [rng.random(int(n)) < p_keep for n in lens]
    return _assemble("tiny", (layers, heads, head_dim), block_size, lens, [None] * requests,
                     keeps, rng, seed)


def llama8b_h2o(seed: int = 0, requests: int = 64, lo: int = 1024, hi: int = 4096,
                layers: int = 32, heads: int = 8, head_dim: int = 128, block_size: int = 16,
                budget_frac: float = 0.2) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    lens = rng.integers(lo, hi + 1, size=requests)
    keeps = []
    for n in lens:
        n = int(n)
        score = rng.lognormal(0.0, 1.5, size=n)
        keeps.append(h2o_mask(np.arange(n), n, score, math.ceil(budget_frac * n)))
    return _assemble("llama8b_h2o", (layers, heads, head_dim), block_size, lens,
                     [None] * requests, keeps, rng, seed)


def mistral7b_random(seed: int = 0, requests: int = 256, lo: int = 512, hi: int = 2048,
                     layers: int = 32, heads: int = 8, head_dim: int = 128, block_size: int = 16,
                     rho_lo: float = 0.3, rho_hi: float = 0.7) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    lens = rng.integers(lo, hi + 1, size=requests)
    rho = rng.uniform(rho_lo, rho_hi, size=requests)
    keeps = [rng.random(int(n)) < rho[r] for r, n in enumerate(lens)]
    return _assemble("mistral7b_random", (layers, heads, head_dim), block_size, lens,
                     [None] * requests, keeps, rng, seed)


def longctx_scissor(seed: int = 0, requests: int = 32, lo: int = 16384, hi: int = 32768,
                    layers: int = 28, heads: int = 4, head_dim: int = 128, block_size: int = 32,
                    n_obs: int = 8, p_hit: float = 0.2, min_hits: int = 2,
                    recent: int = 256) -> Workload:
    """Scissorhands-style: the last ``recent`` tokens stay; an older token stays iff it was
    an importance hit in at least ``min_hits`` of ``n_obs`` observations of the history
    window.  ``n_obs = 8`` (one probe per 64 steps of a 512-step window) keeps about half
    of the tokens; ``n_obs = 512`` is the literal per-step reading, which keeps all."""
    rng = np.random.Generator(np.random.PCG64(seed))
    lens = rng.integers(lo, hi + 1, size=requests)
    keeps = []
    for n in lens:
        n = int(n)
        hits = rng.binomial(n_obs, p_hit, size=n)
        keeps.append((np.arange(n) >= n - recent) | (hits >= min_hits))
    return _assemble("longctx_scissor", (layers, heads, head_dim), block_size, lens,
                     [None] * requests, keeps, rng, seed, notes={"n_obs": n_obs})


def steady_state(seed: int = 0, requests: int = 512, lo: int = 256, hi: int = 8192,
                 layers: int = 32, heads: int = 8, head_dim: int = 128, block_size: int = 16,
                 budget_frac: float = 0.2, thr=(1, 2)) -> Workload:
    """Serving steady state: every request was evicted (H2O-style at length ``len0``) and
    packed once, then grew to ``len``; the mask under test is a second H2O-style eviction pass over
    the resident tokens with the same per-token scores.  Only requests whose live fraction is
    below ``thr`` are repacked (incremental repack)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    lens = rng.integers(lo, hi + 1, size=requests)
    g = rng.uniform(0.5, 1.0, size=requests)
    residents, keeps = [], []
    for r, n in enumerate(lens):
        n = int(n)
        score = rng.lognormal(0.0, 1.5, size=n)
        len0 = int(math.floor(g[r] * n))
        budget0 = max(min(len0, 68), math.ceil(budget_frac * len0))
        surv = np.flatnonzero(h2o_mask(np.arange(len0), len0, score, budget0))
        resident = np.concatenate([surv, np.arange(len0, n)]).astype(np.int64)
        k_res = h2o_mask(resident, n, score, math.ceil(budget_frac * n))
        keep = np.zeros(n, dtype=bool)
        keep[resident[k_res]] = True
        residents.append(resident)
        keeps.append(keep)
    return _assemble("steady_state", (layers, heads, head_dim), block_size, lens, residents,
                     keeps, rng, seed, thr=thr, notes={"g_mean": float(g.mean())})


def streaming_window(seed: int = 0, requests: int = 64, lo: int = 1024, hi: int = 4096, sinks: int = 4,
                     window: int = 512, layers: int = 32, heads: int = 8, head_dim: int = 128,
                     block_size: int = 16) -> Workload:
    """StreamingLLM / sliding-window style mask (Sec. 2.2): the first ``sinks`` tokens (attention
    sinks) and the last ``window`` tokens stay, everything between is evicted.  Whole runs of
    blocks become empty, the sink block and the first window block stay partially live."""
    rng = np.random.Generator(np.random.PCG64(seed))
    lens = rng.integers(lo, hi + 1, size=requests)
    keeps = [(np.arange(int(n)) < sinks) | (np.arange(int(n)) >= int(n) - window) for n in lens]
    return _assemble("streaming_window", (layers, heads, head_dim), block_size, lens, [None] * requests, keeps,
                     rng, seed)


def shared_prefix(seed: int = 0, groups: int = 4, degree: int = 4, prefix_len: int = 8192, suffix_len: int = 8192,
                  layers: int = 32, heads: int = 8, head_dim: int = 128, block_size: int = 16,
                  budget_frac: float = 0.2, extra_free: int = 0):
    """Prefix-cache workload shaped like the paper's compatibility experiment (Sec. 5, Table 1):
    ``groups`` prompts, each shared by ``degree`` requests that reference the SAME physical
    blocks for the first ``prefix_len`` tokens and own a private suffix of ``suffix_len`` tokens;
    H2O-style mask per request over prefix + suffix.  ``prefix_len`` must be a multiple of the
    block size so that shared and private blocks do not mix.  Returns (workload, protect) where
    protect[b] = 1 marks the shared blocks, which a plan must leave in place.  The free list holds
    the destinations of the private suffixes plus 256 blocks; ``extra_free`` adds room for plans that
    copy tokens out of shared blocks as well."""
    S = block_size
    assert prefix_len % S == 0
    rng = np.random.Generator(np.random.PCG64(seed))
    R = groups * degree
    n = prefix_len + suffix_len
    keeps = []
    for r in range(R):
        score = rng.lognormal(0.0, 1.5, size=n)
        keeps.append(h2o_mask(np.arange(n), n, score, math.ceil(budget_frac * n)))
    pre_blocks = prefix_len // S
    suf_blocks = -(-suffix_len // S)
    private_live = [int(k[prefix_len:].sum()) for k in keeps]
    dst_total = sum(-(-x // S) for x in private_live)
    NB = groups * pre_blocks + R * suf_blocks + dst_total + 256 + extra_free
    perm = rng.permutation(NB).astype(np.int32)
    shared = [perm[g * pre_blocks:(g + 1) * pre_blocks] for g in range(groups)]
    cursor = groups * pre_blocks
    bts, tts = [], []
    for r in range(R):
        own = perm[cursor:cursor + suf_blocks]
        cursor += suf_blocks
        blocks = np.concatenate([shared[r // degree], own])
        pos = np.arange(n)
        bts.append(blocks)
        tts.append((blocks[pos // S].astype(np.int64) * S + pos % S).astype(np.int32))
    free_blocks = np.sort(perm[cursor:]).astype(np.int32)
    protect = np.zeros(NB, np.uint8)
    protect[np.concatenate(shared)] = 1
    bt_offsets = np.concatenate([[0], np.cumsum([len(b) for b in bts])]).astype(np.int32)
    tt_offsets = (np.arange(R + 1) * n).astype(np.int32)
    w = Workload(name="shared_prefix", num_layers=layers, num_kv_heads=heads, head_dim=head_dim, block_size=S,
                 num_blocks=NB, bt_offsets=bt_offsets, bt_blocks=np.concatenate(bts).astype(np.int32),
                 tt_offsets=tt_offsets, tt_slots=np.concatenate(tts), keep=np.concatenate(keeps).astype(np.uint8),
                 free_blocks=free_blocks, seed=seed, notes={"degree": degree, "groups": groups,
                                                            "prefix_blocks": pre_blocks})
    return w, protect


CONFIGS = {
    "tiny": tiny,
    "llama8b_h2o": llama8b_h2o,
    "mistral7b_random": mistral7b_random,
    "longctx_scissor": longctx_scissor,
    "steady_state": steady_state,
}


def stats(w: Workload) -> dict:
    """Context statistics of a workload (generator-side description of the INPUT only:
    realised keep fraction, resident tokens, allocated blocks, intra-block waste ratio F of
    Section 2.3.1 before repack, blocks holding at least one kept token)."""
    S = w.block_size
    resident = w.tt_slots >= 0
    kept = resident & (w.keep != 0)
    n_alloc = len(w.bt_blocks)
    per_block = np.bincount(w.tt_slots[kept] // S, minlength=w.num_blocks)
    return {
        "requests": w.num_requests,
        "logical_tokens": w.num_tokens,
        "resident_tokens": int(resident.sum()),
        "kept_tokens": int(kept.sum()),
        "keep_fraction_of_resident": float(kept.sum() / max(1, resident.sum())),
        "allocated_blocks": n_alloc,
        "free_blocks": len(w.free_blocks),
        "num_blocks": w.num_blocks,
        "F_before": float(1.0 - kept.sum() / max(1, n_alloc * S)),
        "blocks_with_a_kept_token": int((per_block > 0).sum()),
        "pool_GiB_k_plus_v": 2 * w.pool_bytes / 2 ** 30,
    }
