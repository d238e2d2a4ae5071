"""TEST INFRASTRUCTURE: CPU plan builder (integer only) - the oracle for ``sched_build``.

The paper gives the scheduler as principles, not as a listing (Section 7.1.2 and the
lessons of Section 7.4.1):

  * one persistent thread block pinned to each SM, processing tasks in a loop;
  * the fixed block-to-SM mapping lets the schedule be planned in advance;
  * each block gets the tasks whose data lives in its SM's local partition (die);
  * data and work are split between the partitions in proportion to their SM counts;
  * the assignment is static;
  * what matters is *which* physical SMs are used, not only how many (Section 1).

Everything more concrete below is this build's reading of those principles, taken
step by step in a fixed order so that the CUDA builder can be compared bytewise.

Work units.  tiles_m = ceil(M / tile_m), tiles_n = ceil(N / tile_n); the K range is cut
into ``k_splits`` runs of whole k-slabs (``k_unit`` elements each).  Unit id
u = (tm * tiles_n + tn) * k_splits + ks.

Steps.
  1. raster order R: tile rows in groups of ``raster_group`` g; inside a group tn is the
     outer loop, tm the middle one, ks the innermost.  g = 1 is the plain row-major raster.
  2. SM set S (ascending), drawn from the SMs not in ``avoid``:
       oblivious, seed 0   the b lowest ids;
       oblivious, seed !=0 Fisher-Yates over the ascending candidate list
                           (i from last down to 1, j = mix64(mix64(seed)+i) mod (i+1)),
                           first b entries, sorted;
       die_compact/affinity  primary die first (preferred_die, else the die with more
                           candidates, tie -> lower id), then the other; inside a die whole
                           TPCs dealt round-robin over that die's GPCs (ascending GPC id,
                           unplaced SMs with gpc < 0 form a last pseudo-GPC), ascending SM id
                           inside a GPC, until b SMs are taken.  With sm_select = 1 ("GPC
                           spread") the dies are not taken one after the other: whole TPCs
                           are dealt round-robin over the GPCs of both dies, which keeps the
                           number of SMs per GPC as low as the budget allows (SMs of one GPC
                           share its port to L2, Section 5.1.2).
                           With cluster_size c > 2 (the kernel to be run launches thread-block clusters of c
                           blocks) the set is built from what can host such clusters: SMs that cluster
                           probing never saw in a cluster larger than 2 ("random" SMs, Section 5.1.1) and
                           unplaced SMs cannot, and a GPC hosts only floor(n / c) clusters on n SMs
                           (Section 7.3: 12 SMs of a GPC form three clusters of 4 but one cluster of 8).
                           In the same die order as above, every GPC's normal candidate SMs (ascending)
                           are cut into blocks of c, an incomplete tail is left aside, and whole blocks
                           are dealt round-robin over the GPCs (block p of every GPC in ascending GPC id,
                           p = 0, 1, ...) while a whole block still fits in the budget.  If the budget is
                           not met that way, it is filled with the normal candidate SMs not yet taken (die
                           order, then ascending id) and last with random and unplaced SMs (same order).
  3. per-die SM counts n_d and rank of each chosen SM inside its die (ascending id).
  4. quotas q_d = floor(n_u * n_d / b); leftover units go one each to the dies in
     descending order of (n_u * n_d mod b), tie -> lower die id.  With die_quota = 1 the dies that
     hold SMs share the units equally instead (weights 1 in place of n_d, their number in place of
     b): for work bound by memory bandwidth over die-local operands, each die's memory being as
     fast as the other's whatever the die's SM count.
  5. unit -> die:
       oblivious    R[i] goes to S[i mod b]; the unit's die is that SM's die;
       die_compact  every raster group (g tile rows) is cut in two in raster order: die 0 takes the
                    first part, die 1 the rest, the cut placed so that after x units of the raster
                    die 0 holds floor(x * q_0 / n_u) of them.  Both dies walk through the raster
                    together and share the row panels of the group they are in, while each keeps its
                    own column panels; with one single group this is two contiguous bands;
       affinity     margin m(u) = local_0(u) - local_1(u) where local_d counts the bytes of
                    the unit's A panel, B panel and C tile that sit in chunks of die d
                    (negated when invert_affinity); a margin with |m| < min_margin counts as 0
                    (in an interleaved layout every unit is about half on each die and the
                    sign of a tiny m is noise); preferred die = 0 if m > 0, 1 if m < 0,
                    the die_compact band's die if m == 0; units sorted by (|m| descending,
                    raster index ascending) are given to their preferred die while its
                    quota lasts, else to the other die; each die's queue is then put back
                    in raster order.
  6. static lists: entry i of die d's queue goes to the SM of rank (i mod n_d) in d.  With
     pair_lists = 1 (plans whose 256-row units are run by the two SMs of a TPC together) the
     entries are dealt to TPCs instead: with P = n_d / 2 TPCs in the die, entry i goes to TPC
     (i mod P) - ranks 2(i mod P) and 2(i mod P)+1 - to its lower SM when (i div P) is even,
     else to its upper SM, so that the two lists of a TPC together hold a fair share of the
     die's work.  (Oblivious plans deal the whole raster the same way over all chosen SMs.)
     Every chosen TPC must be whole and n_d even.
  7. export: flat int32 words (see ``export``).
"""
from __future__ import annotations

import numpy as np

OBLIVIOUS, DIE_COMPACT, AFFINITY = 0, 1, 2
LAYOUT_ROWMAJOR, LAYOUT_PAGED = 0, 1
PLAN_MAGIC = 0x41475031      # "AGP1"
_MASK = (1 << 64) - 1


def mix64(x: int) -> int:
    """The repo's 64-bit mixer, restated here independently of the CUDA side."""
    x = (x + 0x9E3779B97F4A7C15) & _MASK
    x ^= x >> 30
    x = (x * 0xBF58476D1CE4E5B9) & _MASK
    x ^= x >> 27
    x = (x * 0x94D049BB133111EB) & _MASK
    x ^= x >> 31
    return x


def default_policy(**kw) -> dict:
    p = dict(kind=OBLIVIOUS, seed=0, M=0, N=0, K=0, tile_m=128, tile_n=256, k_splits=1,
             k_unit=64, raster_group=1, preferred_die=-1, invert_affinity=0,
             static_assign=1, min_margin=0, sm_select=0, pair_lists=0, cluster_size=1, die_quota=0, avoid=(), a=None, b=None, c=None)
    p.update(kw)
    return p


def operand(offset: int, row_stride: int, elem_bytes: int, layout: int = LAYOUT_ROWMAJOR,
            page_table=None) -> dict:
    return dict(offset=int(offset), row_stride=int(row_stride), elem_bytes=int(elem_bytes),
                layout=layout, page_table=page_table)


# ----------------------------------------------------------------------------- step 1
def raster_order(tiles_m: int, tiles_n: int, k_splits: int, g: int) -> list[int]:
    g = max(1, g)
    R = []
    for tm0 in range(0, tiles_m, g):
        for tn in range(tiles_n):
            for tm in range(tm0, min(tiles_m, tm0 + g)):
                for ks in range(k_splits):
                    R.append((tm * tiles_n + tn) * k_splits + ks)
    return R


# ----------------------------------------------------------------------------- step 2
def select_sms(topo: dict, b: int, pol: dict) -> list[int]:
    n_sm = topo["n_sm"]
    avoid = set(int(s) for s in pol["avoid"])
    cand = [s for s in range(n_sm) if s not in avoid]
    if b < 1 or b > len(cand):
        raise ValueError("sm_budget out of range")
    if pol["kind"] == OBLIVIOUS:
        if pol["seed"] == 0:
            return cand[:b]
        arr = list(cand)
        base = mix64(int(pol["seed"]))
        for i in range(len(arr) - 1, 0, -1):
            j = mix64((base + i) & _MASK) % (i + 1)
            arr[i], arr[j] = arr[j], arr[i]
        return sorted(arr[:b])
    die, gpc, tpc = topo["die"], topo["gpc"], topo["tpc"]
    n_gpc = topo["n_gpc"]
    cnt = [sum(1 for s in cand if die[s] == d) for d in (0, 1)]
    if pol["preferred_die"] in (0, 1):
        primary = pol["preferred_die"]
    else:
        primary = 0 if cnt[0] >= cnt[1] else 1
    S = []
    die_passes = [(0, 1)] if pol.get("sm_select", 0) == 1 else [(primary,), (1 - primary,)]
    csize = int(pol.get("cluster_size", 1))
    if csize > 2:
        rnd = topo["is_random"]
        normal = lambda s: (not rnd[s]) and gpc[s] >= 0
        for dies in die_passes:
            per_gpc: dict[int, list[int]] = {}
            for s in cand:
                if die[s] in dies and normal(s):
                    per_gpc.setdefault(int(gpc[s]), []).append(s)
            keys = sorted(per_gpc)
            blocks = {k: [per_gpc[k][i:i + csize] for i in range(0, len(per_gpc[k]) - csize + 1, csize)] for k in keys}
            p = 0
            while any(p < len(blocks[k]) for k in keys):
                for k in keys:
                    if p < len(blocks[k]) and len(S) + csize <= b:
                        S += blocks[k][p]
                p += 1
        chosen = set(S)
        for want_normal in (True, False):
            for dies in die_passes:
                for s in cand:
                    if len(S) < b and s not in chosen and die[s] in dies and normal(s) == want_normal:
                        S.append(s)
                        chosen.add(s)
        return sorted(S)
    for dies in die_passes:
        # candidate TPCs of these dies, grouped by GPC key (gpc < 0 -> pseudo-GPC n_gpc)
        groups: dict[int, dict[int, list[int]]] = {}
        for s in cand:
            if die[s] not in dies:
                continue
            key = int(gpc[s]) if gpc[s] >= 0 else n_gpc
            groups.setdefault(key, {}).setdefault(int(tpc[s]), []).append(s)
        keys = sorted(groups)
        lists = {k: [groups[k][t] for t in sorted(groups[k])] for k in keys}
        p = 0
        while len(S) < b and any(p < len(lists[k]) for k in keys):
            for k in keys:
                if p < len(lists[k]):
                    for s in lists[k][p]:
                        if len(S) < b:
                            S.append(s)
            p += 1
        if len(S) >= b:
            break
    return sorted(S)


def cluster_capacity(topo: dict, S, csize: int) -> int:
    """Thread-block clusters of ``csize`` blocks that the SM set S can host at once, one block per SM: per GPC,
    floor(normal SMs of S in it / csize); random and unplaced SMs host none when csize > 2 (Sections 5.1.1, 7.3)."""
    per = {}
    for s in S:
        if csize > 2 and (topo["is_random"][s] or topo["gpc"][s] < 0):
            continue
        key = int(topo["gpc"][s]) if topo["gpc"][s] >= 0 else -1 - int(s) // 2      # unplaced: only its own TPC
        per[key] = per.get(key, 0) + 1
    return sum(n // csize for n in per.values())


# ----------------------------------------------------------------------------- step 4
def quotas(n_u: int, n_d: list[int], b: int) -> list[int]:
    q = [n_u * n // b for n in n_d]
    rem = [n_u * n % b for n in n_d]
    left = n_u - sum(q)
    order = sorted(range(len(n_d)), key=lambda d: (-rem[d], d))
    for d in order:
        if left == 0:
            break
        if n_d[d] > 0:
            q[d] += 1
            left -= 1
    assert left == 0
    return q


# ----------------------------------------------------------------------------- step 5 helpers
def band_die(i: int, n_u: int, q0: int, group_len: int) -> int:
    """Die that the die_compact rule gives raster index i (see step 5)."""
    start = (i // group_len) * group_len
    end = min(n_u, start + group_len)
    cut = (end * q0) // n_u - (start * q0) // n_u       # die-0 units inside this raster group
    return 0 if i - start < cut else 1



def k_range(pol: dict, ks: int) -> tuple[int, int]:
    """Element range [k0, k1) of split ks: whole k-slabs, the first splits take the longer runs."""
    K, ku = pol["K"], pol["k_unit"]
    n_slab = -(-K // ku)
    per = -(-n_slab // pol["k_splits"])
    s0 = min(n_slab, ks * per)
    s1 = min(n_slab, (ks + 1) * per)
    return min(K, s0 * ku), min(K, s1 * ku)


def _bytes_per_die_interval(amap: dict, start: int, end: int) -> list[int]:
    """Bytes of [start, end) (offsets from the probed base) that lie in chunks of die 0 / 1."""
    cb = amap["chunk_bytes"]
    doc = amap["die_of_chunk"]
    out = [0, 0]
    pos = start
    while pos < end:
        c = pos // cb
        nxt = min(end, (c + 1) * cb)
        out[int(doc[c])] += nxt - pos
        pos = nxt
    return out


def unit_local_bytes(pol: dict, amap: dict, u: int) -> list[int]:
    """local_d(u): bytes of unit u's A panel, B panel and C tile in chunks of die d."""
    tiles_n = -(-pol["N"] // pol["tile_n"])
    ks = u % pol["k_splits"]
    t = u // pol["k_splits"]
    tm, tn = t // tiles_n, t % tiles_n
    r0, r1 = tm * pol["tile_m"], min(pol["M"], (tm + 1) * pol["tile_m"])
    c0, c1 = tn * pol["tile_n"], min(pol["N"], (tn + 1) * pol["tile_n"])
    k0, k1 = k_range(pol, ks)
    tot = [0, 0]

    def add(op, row_lo, row_hi, col_lo, col_hi):
        if op is None:
            return
        eb = op["elem_bytes"]
        for r in range(row_lo, row_hi):
            s = op["offset"] + r * op["row_stride"] + col_lo * eb
            e = op["offset"] + r * op["row_stride"] + col_hi * eb
            v = _bytes_per_die_interval(amap, s, e)
            tot[0] += v[0]
            tot[1] += v[1]

    add(pol["a"], r0, r1, k0, k1)                      # A panel: rows of the tile, k-range columns
    bop = pol["b"]
    if bop is not None and bop["layout"] == LAYOUT_PAGED:
        # weights stored as 4 KB pages of [128 columns x 16 k] elements; logical page of
        # (128-column block pc, k16) = pc * ceil(K/16) + k16; a unit column holds tile_n/128 blocks
        ppt = -(-pol["K"] // 16)
        ppc = max(1, pol["tile_n"] // 128)
        cb = amap["chunk_bytes"]
        for pc in range(tn * ppc, (tn + 1) * ppc):
            for k16 in range(k0 // 16, -(-k1 // 16)):
                phys = int(bop["page_table"][pc * ppt + k16])
                tot[int(amap["die_of_chunk"][phys])] += cb
    else:
        add(bop, k0, k1, c0, c1)                       # B panel: k-range rows, tile columns
    add(pol["c"], r0, r1, c0, c1)                      # C tile
    return tot


# ----------------------------------------------------------------------------- whole plan
def build_plan(topo: dict, amap: dict | None, b: int, pol: dict) -> dict:
    M, N, K = pol["M"], pol["N"], pol["K"]
    tiles_m = -(-M // pol["tile_m"])
    tiles_n = -(-N // pol["tile_n"])
    ksp = pol["k_splits"]
    n_u = tiles_m * tiles_n * ksp
    R = raster_order(tiles_m, tiles_n, ksp, pol["raster_group"])
    S = select_sms(topo, b, pol)
    die = topo["die"]
    sm_die = [int(die[s]) for s in S]
    n_d = [sm_die.count(0), sm_die.count(1)]
    rank = []
    seen = [0, 0]
    for d in sm_die:
        rank.append(seen[d])
        seen[d] += 1
    slots_of_die = [[i for i, d in enumerate(sm_die) if d == dd] for dd in (0, 1)]
    if pol.get("die_quota", 0):
        w = [1 if n > 0 else 0 for n in n_d]
        q = quotas(n_u, w, sum(w))
    else:
        q = quotas(n_u, n_d, b)

    sm_q = [[] for _ in S]
    pair_lists = pol.get("pair_lists", 0)
    if pair_lists:
        tpc = topo["tpc"]
        groups = [list(range(b))] if pol["kind"] == OBLIVIOUS else slots_of_die
        for slots in groups:
            if len(slots) % 2 or any(tpc[S[slots[2 * j]]] != tpc[S[slots[2 * j + 1]]] for j in range(len(slots) // 2)):
                raise ValueError("pair_lists needs whole TPCs")

    def pair_slot(slots, i):
        P = len(slots) // 2
        return slots[2 * (i % P) + ((i // P) & 1)]

    if pol["kind"] == OBLIVIOUS:
        die_q = [[], []]
        for i, u in enumerate(R):
            slot = pair_slot(list(range(b)), i) if pair_lists else i % b
            sm_q[slot].append(u)
            die_q[sm_die[slot]].append(u)
    else:
        group_len = max(1, pol["raster_group"]) * tiles_n * ksp
        if pol["kind"] == DIE_COMPACT:
            die_q = [[], []]
            for i, u in enumerate(R):
                die_q[band_die(i, n_u, q[0], group_len)].append(u)
        else:
            if amap is None:
                raise ValueError("affinity policy needs an affinity map")
            items = []
            for i, u in enumerate(R):
                l0, l1 = unit_local_bytes(pol, amap, u)
                m = l0 - l1
                if pol["invert_affinity"]:
                    m = -m
                if abs(m) < pol["min_margin"]:
                    m = 0
                if m > 0:
                    pref = 0
                elif m < 0:
                    pref = 1
                else:
                    pref = band_die(i, n_u, q[0], group_len)
                items.append((-abs(m), i, u, pref))
            items.sort()
            got = [[], []]
            for _, i, u, pref in items:
                d = pref if len(got[pref]) < q[pref] else 1 - pref
                got[d].append((i, u))
            die_q = [[u for _, u in sorted(g)] for g in got]
        for d in (0, 1):
            for i, u in enumerate(die_q[d]):
                slot = pair_slot(slots_of_die[d], i) if pair_lists else slots_of_die[d][i % n_d[d]]
                sm_q[slot].append(u)

    smid_to_slot = [-1] * topo["n_sm"]
    for i, s in enumerate(S):
        smid_to_slot[s] = i
    return dict(kind=pol["kind"], n_sm=topo["n_sm"], b=b, n_units=n_u, tiles_m=tiles_m,
                tiles_n=tiles_n, k_splits=ksp, tile_m=pol["tile_m"], tile_n=pol["tile_n"],
                M=M, N=N, K=K, static_assign=pol["static_assign"],
                sm_list=S, sm_die=sm_die, rank_in_die=rank, die_sm_count=n_d,
                die_q=die_q, sm_q=sm_q, smid_to_slot=smid_to_slot, quotas=q)


def export(plan: dict) -> np.ndarray:
    """Flat int32 image compared bytewise with the library's ``ag_plan_export``:

    header[16] = magic, kind, n_sm, b, n_die(2), n_units, tiles_m, tiles_n, k_splits,
                 tile_m, tile_n, M, N, K, static_assign, 0
    then sm_list[b], sm_die[b], rank_in_die[b], die_sm_count[2], die_q_off[3],
    die_q[n_units], sm_q_off[b+1], sm_q[n_units], smid_to_slot[n_sm].
    """
    p = plan
    w = [PLAN_MAGIC, p["kind"], p["n_sm"], p["b"], 2, p["n_units"], p["tiles_m"], p["tiles_n"],
         p["k_splits"], p["tile_m"], p["tile_n"], p["M"], p["N"], p["K"], p["static_assign"], 0]
    w += p["sm_list"] + p["sm_die"] + p["rank_in_die"] + p["die_sm_count"]
    w += [0, len(p["die_q"][0]), len(p["die_q"][0]) + len(p["die_q"][1])]
    w += p["die_q"][0] + p["die_q"][1]
    off = [0]
    for lst in p["sm_q"]:
        off.append(off[-1] + len(lst))
    w += off
    for lst in p["sm_q"]:
        w += lst
    w += p["smid_to_slot"]
    return np.array(w, dtype=np.int32)


# ----------------------------------------------------------------------------- die-view packing
def build_page_table(page_die, amap: dict) -> list[int]:
    """Indirect allocation by remapping (Section 7.1.1, Eq. 1 of the remapping appendix).

    The packed buffer is read as aligned pairs of 4 KB chunks (2p, 2p+1); by the pair rule one
    chunk of every pair sits on each die.  Two logical views are laid over the buffer, one per die:
    page p of view d is the chunk of pair p that sits on die d.  Logical weight page j (owned by a
    work unit that the plan gave to die ``page_die[j]``) takes the next free page of that die's
    view.  The measured chunk->die bit replaces the parity-of-masked-physical-address selector of
    Eq. 1, which needs a physical base address that an unmodified driver does not expose.
    Where a pair has both chunks on one die x (the pair rule fails), view x takes the even chunk
    and the other view the odd one, so that no chunk is used twice.
    """
    doc = amap["die_of_chunk"]
    nxt = [0, 0]
    table = []
    for d in page_die:
        d = int(d)
        pair = nxt[d]
        nxt[d] += 1
        # even chunk if it sits on die d, else the odd one (also right when the pair rule fails:
        # both chunks on die x -> view x gets the even chunk, the other view the odd one)
        table.append(2 * pair + (0 if int(doc[2 * pair]) == d else 1))
    return table


def quad_groups(amap: dict, free_bit: int, first: int = 0) -> list[list[int]]:
    """Groups of four chunks that an XOR partition hash (Section 6.1.2) keeps on one die when chunk-index
    bits 0 and 1 take part in it and bit ``free_bit`` (>= 2) does not: flipping bits 0 and 1 together, or the
    free bit, leaves the parity unchanged.  With F = 2**free_bit the groups are
        {q, q+3, q+F, q+F+3}   for q = 0 (mod 4)   and   {q, q+1, q+F, q+F+1}   for q = 1 (mod 4),
    q with bit ``free_bit`` clear.  The hash works on addresses, so the bit tests are made on first + q, where
    ``first`` is the chunk index of the buffer's base inside its 2 MiB page (0 for an aligned buffer); q itself is
    relative to the buffer.  Returned per die, in ascending q, as [die0 bases, die1 bases]; a group whose four
    measured chunks do not agree (noise) is left out.
    """
    doc = amap["die_of_chunk"]
    n = len(doc)
    F = 1 << free_bit
    out = [[], []]
    for q in range(n):
        qa = first + q
        if (qa & F) or (qa & 3) > 1:
            continue
        a = 3 if (qa & 3) == 0 else 1
        members = [q, q + a, q + F, q + F + a]
        if members[-1] >= n:
            continue
        dies = {int(doc[c]) for c in members}
        if len(dies) == 1:
            out[dies.pop()].append(q)
    return out


def build_page_table_quads(page_die, amap: dict, free_bit: int, first: int = 0) -> list[int]:
    """Page table when the packed weights are laid out in groups of four chunks (one k-slab of a 128-column
    block = four 4 KB pages = one group, fetched by a single strided copy).  Logical pages come in runs of four
    (k16 = 4s .. 4s+3) owned by one die; run number r of die d takes the r-th group of that die's view and its
    pages go to the group's chunks in the order q, q+a, q+F, q+F+a."""
    groups = quad_groups(amap, free_bit, first)
    F = 1 << free_bit
    nxt = [0, 0]
    table = []
    assert len(page_die) % 4 == 0
    for r in range(len(page_die) // 4):
        d = int(page_die[4 * r])
        assert all(int(x) == d for x in page_die[4 * r:4 * r + 4])
        q = groups[d][nxt[d]]
        nxt[d] += 1
        a = 3 if ((first + q) & 3) == 0 else 1
        table += [q, q + a, q + F, q + F + a]
    return table


def _parity(x: int) -> int:
    return bin(x).count("1") & 1


def fit_page_constants(amap: dict, mask: int, first: int = 0) -> tuple[list[int], int]:
    """The part of the partition hash (Section 6.1.2) that the in-page mask does not explain: one bit per 2 MiB
    page (512 chunks; pages are counted in first + q, ``first`` = chunk index of the buffer's base inside its
    page), taken as the majority of die ^ parity((first + q) & mask) over the page's chunks.  Returns the bits
    and the number of chunks that disagree with parity ^ bit (noise, or a layout that is no such hash)."""
    doc = amap["die_of_chunk"]
    n = len(doc)
    n_pages = (first + n + 511) // 512
    ones = [0] * n_pages
    cnt = [0] * n_pages
    for q in range(n):
        qa = first + q
        ones[qa >> 9] += int(doc[q]) ^ _parity(qa & mask)
        cnt[qa >> 9] += 1
    bits = [1 if 2 * ones[i] > cnt[i] else 0 for i in range(n_pages)]
    bad = sum(1 for q in range(n) if (int(doc[q]) ^ _parity((first + q) & mask)) != bits[(first + q) >> 9])
    return bits, bad


def page_from_hash(j: int, P: int, mask: int, c_bits, first: int = 0) -> int:
    """Eq. 1 of the remapping appendix in closed form: logical page j of the view of die P is the chunk of the
    aligned pair (2j, 2j+1) that the hash places on die P,
        chunk = 2j + (parity((first + 2j) & mask) ^ c_page ^ P),
    with the measured in-page mask standing for MASK and the per-2-MiB-page bit c_page for what the address bits
    above bit 20 contribute.  Needs chunk-index bit 0 in the mask and an even ``first`` (aligned pairs)."""
    qa = first + 2 * j
    return 2 * j + (_parity(qa & mask) ^ int(c_bits[qa >> 9]) ^ P)


def quad_group_from_hash(r: int, d: int, mask: int, c_bits, free_bit: int, first: int = 0) -> tuple[int, int]:
    """The r-th group of four same-die chunks (see ``quad_groups``) of die d, in ascending order of its base chunk,
    without a table: (base chunk q relative to the buffer, a).  With F = 2**free_bit, every run of four chunks
    4t .. 4t+3 (absolute index first + q, bit ``free_bit`` clear) holds one group base per die - chunk 4t if
    parity(4t & mask) ^ c_page is d (then a = 3), else chunk 4t + 1 (a = 1) - so the r-th group of either die sits in
    the r-th such run at or after ``first``.  Needs bits 0 and 1 in the mask, bit ``free_bit`` out of it, and
    ``first`` a multiple of 4."""
    F = 1 << free_bit

    def runs_below(x):                    # runs 4t..4t+3 with bit free_bit clear that start below absolute chunk x
        return (x // (2 * F)) * (F // 4) + min(x % (2 * F), F) // 4
    T = r + runs_below(first)
    qa0 = (T // (F // 4)) * 2 * F + (T % (F // 4)) * 4
    e = _parity(qa0 & mask) ^ int(c_bits[qa0 >> 9]) ^ d
    return qa0 + e - first, (3 if e == 0 else 1)


def page_die_from_plan(plan: dict, K: int, k_unit: int = 64) -> list[int]:
    """Die that owns every logical weight page (pc, k16), j = pc * ceil(K/16) + k16, pc = index of the
    128-column block: the die whose queue holds most of the units (tm, tn, ks) that read the page
    (tn = pc // (tile_n/128), ks = the k-split containing k16; a tie goes to die 0).  Decode-shaped
    plans have one tile row, so exactly one unit reads a page."""
    unit_die = {}
    for d in (0, 1):
        for u in plan["die_q"][d]:
            unit_die[u] = d
    ksp, tiles_m, tiles_n = plan["k_splits"], plan["tiles_m"], plan["tiles_n"]
    n_slab = -(-K // k_unit)
    per = -(-n_slab // ksp)
    ppt = -(-K // 16)
    ppc = max(1, plan["tile_n"] // 128)
    out = []
    for pc in range(tiles_n * ppc):
        tn = pc // ppc
        for k16 in range(ppt):
            ks = (k16 * 16 // k_unit) // per
            votes = [0, 0]
            for tm in range(tiles_m):
                votes[unit_die[(tm * tiles_n + tn) * ksp + ks]] += 1
            out.append(0 if votes[0] >= votes[1] else 1)
    return out


def pack_weights(B_bits: np.ndarray, page_table: list[int], n_chunks: int, tile_n: int = 128) -> np.ndarray:
    """Packed image (uint16, n_chunks x 2048) of the K x N bf16 weights (tile_n = page width, 128).

    Logical page (pc, k16) holds W[n][k] for n in [pc*128, pc*128+128), k in [k16*16, k16*16+16)
    as 8 x 8 blocks ("core matrices", 8 rows n x 16 bytes of k, 128 bytes each, row-major inside):
    element (n, k) of the page sits at byte (n//8)*256 + (k//8)*128 + (n%8)*16 + (k%8)*2.
    Out-of-range n or k are zeros; chunks no page maps to stay zero.
    """
    K, N = B_bits.shape
    ppt = -(-K // 16)
    tiles_n = -(-N // tile_n)
    out = np.zeros((n_chunks, 2048), dtype=np.uint16)
    for tn in range(tiles_n):
        for k16 in range(ppt):
            page = np.zeros((tile_n, 16), dtype=np.uint16)
            k0, n0 = k16 * 16, tn * tile_n
            blk = B_bits[k0:min(K, k0 + 16), n0:min(N, n0 + tile_n)]       # [k][n]
            page[:blk.shape[1], :blk.shape[0]] = blk.T
            # (n//8, n%8, k//8, k%8) -> (n//8, k//8, n%8, k%8)
            img = page.reshape(tile_n // 8, 8, 2, 8).transpose(0, 2, 1, 3).reshape(-1)
            out[page_table[tn * ppt + k16]] = img
    return out
