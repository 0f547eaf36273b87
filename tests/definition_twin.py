"""A second, definition-level statement of the repack result in pure Python containers
(lists, dicts, sets), used only to brute-force the C oracle on tiny inputs.

It is organised differently from the C oracle on purpose: it first collects the facts about
every request, then decides admission for all of them at once from the running demand, then
builds the outputs from per-request dictionaries.  Statuses: 0 not selected, 1 repacked,
2 no gain, 3 deferred.
"""
from fractions import Fraction
from itertools import accumulate


def repack_definition(S, block_tables, token_tables, keeps, free, select=None, thr=None):
    """block_tables[r]: list of block ids; token_tables[r]: list of slot or -1;
    keeps[r]: list of 0/1; free: list of block ids; thr: Fraction or None.
    Returns dict(new_bt, new_tt, freed, status, moves, consumed)."""
    R = len(token_tables)
    live = [[t for t, (s, k) in enumerate(zip(token_tables[r], keeps[r])) if s >= 0 and k]
            for r in range(R)]
    need = [-(-len(live[r]) // S) for r in range(R)]

    def chosen(r):
        if select is not None and not select[r]:
            return False
        if thr is not None:
            capacity = len(block_tables[r]) * S
            # live fraction strictly below the threshold; a request with no blocks never is
            if capacity == 0 or not Fraction(len(live[r]), capacity) < thr:
                return False
        return True

    candidates = [r for r in range(R) if chosen(r) and need[r] < len(block_tables[r])]
    running = list(accumulate(need[r] for r in candidates))
    fits = [c <= len(free) for c in running]
    n_admit = fits.index(False) if False in fits else len(candidates)
    admitted = candidates[:n_admit]
    deferred = set(candidates[n_admit:])

    status = []
    for r in range(R):
        if r in admitted:
            status.append(1)
        elif r in deferred:
            status.append(3)
        elif chosen(r):
            status.append(2)
        else:
            status.append(0)

    cursor = 0
    new_bt, new_tt, freed, moves = [], [], [], []
    for r in range(R):
        if r in admitted:
            mine = free[cursor:cursor + need[r]]
            cursor += need[r]
            where = {t: mine[i // S] * S + i % S for i, t in enumerate(live[r])}
            new_bt.append(list(mine))
            freed.extend(block_tables[r])
            moves.extend((token_tables[r][t], where[t]) for t in live[r])
        else:
            where = {t: token_tables[r][t] for t in live[r]}
            new_bt.append(list(block_tables[r]))
        new_tt.append([where.get(t, -1) for t in range(len(token_tables[r]))])
    return dict(new_bt=new_bt, new_tt=new_tt, freed=freed, status=status, moves=moves,
                consumed=cursor)


def to_csr(lists):
    offsets = [0]
    flat = []
    for x in lists:
        flat.extend(x)
        offsets.append(len(flat))
    return offsets, flat


def repack_partial_definition(S, block_tables, token_tables, keeps, free, select=None, thr=None, protect=(),
                              util=None, max_sources=0, theta=None, detach=None, detach_rule=0):
    """Definition-level statement of the partial plan: only low-utilisation, unprotected blocks are
    evacuated.  protect: set of block ids; util / theta / detach: Fraction or None.  With ``detach`` a
    request whose own live tokens fill less than that fraction of its protected blocks leaves all of
    them (copy-on-write): they become sources too and are listed under ``released``.  With
    ``detach_rule`` 1 the fraction is taken block by block: the request leaves exactly the protected
    blocks in which its own live tokens fill less than ``detach`` of the S slots; with 2 the block is
    judged by the live tokens of all requests stored in it."""
    R = len(token_tables)
    live = [[t for t, (s, k) in enumerate(zip(token_tables[r], keeps[r])) if s >= 0 and k] for r in range(R)]
    per_block = {}
    for r in range(R):
        for t in live[r]:
            b = token_tables[r][t] // S
            per_block[b] = per_block.get(b, 0) + 1
    allocated = sum(len(b) for b in block_tables)
    total_live = sum(len(x) for x in live)
    triggered = True
    if theta is not None:
        triggered = allocated > 0 and 1 - Fraction(total_live, allocated * S) > theta

    sources, leaving = [], []
    for r in range(R):
        picked = []
        for b in block_tables[r]:
            ok = b not in protect and (util is None or Fraction(per_block.get(b, 0), S) < util)
            if ok and (max_sources == 0 or len(picked) < max_sources):
                picked.append(b)
        shared = [b for b in block_tables[r] if b in protect]
        mine_in_shared = sum(1 for t in live[r] if token_tables[r][t] // S in protect)
        if detach is not None and detach_rule == 1:
            mine_in = lambda b: sum(1 for t in live[r] if token_tables[r][t] // S == b)
            leaving.append({b for b in shared if Fraction(mine_in(b), S) < detach})
        elif detach is not None and detach_rule == 2:
            leaving.append({b for b in shared if Fraction(per_block.get(b, 0), S) < detach})
        else:
            goes = detach is not None and shared and Fraction(mine_in_shared, len(shared) * S) < detach
            leaving.append(set(shared) if goes else set())
        # table order is kept: a source is an unprotected pick or a shared block of a leaving request
        sources.append([b for b in block_tables[r] if b in set(picked) or b in leaving[r]])
    moving = [[t for t in live[r] if token_tables[r][t] // S in set(sources[r])] for r in range(R)]
    need = [-(-len(moving[r]) // S) for r in range(R)]

    def chosen(r):
        if not triggered or (select is not None and not select[r]):
            return False
        if thr is not None:
            capacity = len(block_tables[r]) * S
            if capacity == 0 or not Fraction(len(live[r]), capacity) < thr:
                return False
        return True

    candidates = [r for r in range(R) if chosen(r) and need[r] < len(sources[r])]
    running = list(accumulate(need[r] for r in candidates))
    fits = [c <= len(free) for c in running]
    n_admit = fits.index(False) if False in fits else len(candidates)
    admitted, deferred = candidates[:n_admit], set(candidates[n_admit:])
    status = [1 if r in admitted else 3 if r in deferred else 2 if chosen(r) else 0 for r in range(R)]

    cursor = 0
    new_bt, new_tt, freed, released, moves = [], [], [], [], []
    for r in range(R):
        where = {t: token_tables[r][t] for t in live[r]}
        if r in admitted:
            mine = free[cursor:cursor + need[r]]
            cursor += need[r]
            for i, t in enumerate(moving[r]):
                where[t] = mine[i // S] * S + i % S
                moves.append((token_tables[r][t], where[t]))
            src = set(sources[r])
            new_bt.append([b for b in block_tables[r] if b not in src] + list(mine))
            freed.extend(b for b in block_tables[r] if b in src and b not in leaving[r])
            released.extend(b for b in block_tables[r] if b in leaving[r])
        else:
            new_bt.append(list(block_tables[r]))
        new_tt.append([where.get(t, -1) for t in range(len(token_tables[r]))])
    return dict(new_bt=new_bt, new_tt=new_tt, freed=freed, released=released, status=status, moves=moves,
                consumed=cursor)
