"""Seeded synthetic inputs: programs in CSR form and per-operand candidate rows.

This module only *builds inputs*.  It contains no liveness analysis and no
verification logic: every live interval it uses is known from how the program
was constructed (who reads which value, and which loops enclose the reader), so
its "valid" rows are valid by construction and serve as an independent check of
both the CPU oracle and the CUDA path.

Program model (stands in for the paper's GEMM / attention machine-IR corpus,
Section 4.1, which is not redistributable):

* blocks are laid out in an order in which every block follows its dominators;
  loops are contiguous block ranges;
* every instruction defines exactly one virtual register and reads 0..3 values
  ("uses by geometric recency": a read reaches back G ~ Geom(0.3) positions in
  the list of values that are visible and not yet overwritten);
* short-lived virtual registers are drawn from a per-block pool and re-defined
  cyclically, so a vreg has several definitions (post-phi machine IR, not SSA);
* loop-carried accumulators are defined once before their loop, updated by
  ``acc = op(acc, x, y)`` instructions spread through the loop blocks and read
  once after the loop;
* a candidate row holds one uint16 physical register per operand occurrence.

Random numbers come from a counter-based generator (splitmix64 finaliser over
(seed, stream, index)), so any element can be regenerated independently and the
result does not depend on numpy's generators.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Sequence, Tuple

import numpy as np

U64 = np.uint64
_MASK64 = (1 << 64) - 1
_GOLD = 0x9E3779B97F4A7C15

# random streams
_S_WIDTH, _S_UCOUNT, _S_GEOM, _S_PERM, _S_XOR, _S_FAULT, _S_FKIND, _S_FPICK, _S_SHAPE = range(1, 10)

KIND_NORMAL, KIND_ACC_DEF, KIND_ACC_UPD, KIND_ACC_READ = 0, 1, 2, 3

FAULT_NONE, FAULT_INCONSISTENT, FAULT_OVERLAP, FAULT_RANGE = 0, 1, 2, 3


# --------------------------------------------------------------------------- rng
def _mix(z: np.ndarray) -> np.ndarray:
    z = z.astype(U64, copy=True)
    z ^= z >> U64(30)
    z *= U64(0xBF58476D1CE4E5B9)
    z ^= z >> U64(27)
    z *= U64(0x94D049BB133111EB)
    z ^= z >> U64(31)
    return z


def rnd_u64(seed: int, stream: int, idx) -> np.ndarray:
    """64 random bits for every index; a pure function of (seed, stream, idx)."""
    idx = np.atleast_1d(np.asarray(idx)).astype(U64)
    key = ((seed & _MASK64) * _GOLD + (stream & _MASK64) * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D) & _MASK64
    key = _mix(np.array([key], dtype=U64))
    return _mix(key + idx * U64(_GOLD))


def rnd_unit(seed: int, stream: int, idx) -> np.ndarray:
    """Uniform doubles in [0, 1)."""
    return (rnd_u64(seed, stream, idx) >> U64(11)).astype(np.float64) * (1.0 / (1 << 53))


# ------------------------------------------------------------------------ shapes
@dataclass
class AccGroup:
    count: int
    def_block: int
    update_blocks: Tuple[int, ...]
    read_block: int


@dataclass
class Shape:
    name: str
    block_sizes: List[int]
    edges: List[Tuple[int, int]]
    loops: List[Tuple[int, int]]          # inclusive block ranges
    acc_groups: List[AccGroup]
    n_vregs: int
    widths: Dict[int, float]
    P: int
    B: int = 4


@dataclass
class Program:
    """CSR program, field for field what the C ABI's program descriptor holds."""
    n_blocks: int
    n_instrs: int
    n_vregs: int
    n_operands: int
    n_edges: int
    P: int
    B: int
    block_instr_off: np.ndarray   # u32 [n_blocks+1]
    succ_off: np.ndarray          # u32 [n_blocks+1]
    succ: np.ndarray              # u32 [n_edges]
    instr_op_off: np.ndarray      # u32 [n_instrs+1]
    instr_n_defs: np.ndarray      # u8  [n_instrs]
    op_vreg: np.ndarray           # u32 [n_operands]
    vreg_width: np.ndarray        # u8  [n_vregs]
    gen: dict = field(default_factory=dict)   # construction bookkeeping (not part of the ABI)

    @property
    def pitch(self) -> int:
        """Row pitch in elements: operand count rounded up to 8 (16-byte rows)."""
        return max(8, (self.n_operands + 7) // 8 * 8)


def program_from_lists(blocks, edges, n_vregs, widths, P, B=4) -> Program:
    """Hand-built program.  ``blocks`` is a list of blocks, each a list of
    instructions ``(defs, uses)`` with vreg ids; ``edges`` a list of (from, to)."""
    nB = len(blocks)
    blk_off = [0]
    op_off = [0]
    n_defs = []
    ops = []
    for blk in blocks:
        for defs, uses in blk:
            ops.extend(defs)
            ops.extend(uses)
            n_defs.append(len(defs))
            op_off.append(len(ops))
        blk_off.append(len(n_defs))
    succ_lists = [[] for _ in range(nB)]
    for a, b in edges:
        succ_lists[a].append(b)
    succ_off = [0]
    succ = []
    for s in succ_lists:
        succ.extend(s)
        succ_off.append(len(succ))
    return Program(
        n_blocks=nB, n_instrs=len(n_defs), n_vregs=n_vregs, n_operands=len(ops), n_edges=len(succ),
        P=P, B=B,
        block_instr_off=np.array(blk_off, dtype=np.uint32),
        succ_off=np.array(succ_off, dtype=np.uint32),
        succ=np.array(succ, dtype=np.uint32),
        instr_op_off=np.array(op_off, dtype=np.uint32),
        instr_n_defs=np.array(n_defs, dtype=np.uint8),
        op_vreg=np.array(ops, dtype=np.uint32),
        vreg_width=np.array(widths, dtype=np.uint8),
    )


# ------------------------------------------------------------------ program build
def _dominator_chains(nB: int, edges: Sequence[Tuple[int, int]]) -> List[List[int]]:
    """Strict dominators of every block, nearest first (plain iterative sets)."""
    preds = [[] for _ in range(nB)]
    for a, b in edges:
        preds[b].append(a)
    full = set(range(nB))
    dom = [set(full) for _ in range(nB)]
    dom[0] = {0}
    changed = True
    while changed:
        changed = False
        for b in range(1, nB):
            ps = [dom[p] for p in preds[b]]
            new = (set.intersection(*ps) if ps else set()) | {b}
            if new != dom[b]:
                dom[b] = new
                changed = True
    chains = []
    for b in range(nB):
        strict = [d for d in dom[b] if d != b]
        strict.sort(key=lambda d: -len(dom[d]))
        chains.append(strict)
    return chains


def _largest_remainder(total: int, weights: np.ndarray, caps: np.ndarray) -> np.ndarray:
    """Split ``total`` proportionally to ``weights`` with 1 <= part <= cap where cap > 0."""
    w = weights.astype(np.float64)
    out = np.zeros(len(w), dtype=np.int64)
    live = caps > 0
    if total < live.sum():
        raise ValueError("fewer pool vregs than blocks that need one")
    quota = w / w[live].sum() * total
    out[live] = np.clip(np.floor(quota[live]).astype(np.int64), 1, caps[live])
    # hand out / take back the remainder, largest fractional part first
    for _ in range(4 * len(w) + 4 * abs(int(total - out.sum())) + 8):
        diff = total - int(out.sum())
        if diff == 0:
            break
        frac = quota - out
        if diff > 0:
            cand = np.where(live & (out < caps))[0]
            if len(cand) == 0:
                raise ValueError("vreg pools do not fit the blocks")
            j = cand[np.argmax(frac[cand])]
            out[j] += 1
        else:
            cand = np.where(live & (out > 1))[0]
            j = cand[np.argmin(frac[cand])]
            out[j] -= 1
    if out.sum() != total:
        raise ValueError("vreg pools do not fit the blocks")
    return out


def make_program(shape: Shape, seed: int) -> Program:
    nB = len(shape.block_sizes)
    sizes = np.asarray(shape.block_sizes, dtype=np.int64)
    blk_off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    nI = int(blk_off[-1])
    blk_of = np.repeat(np.arange(nB), sizes)

    # ---- instruction kinds: accumulator definitions / updates / reads, evenly spread
    kind = np.zeros(nI, dtype=np.int8)
    acc_of = np.full(nI, -1, dtype=np.int64)
    n_acc = sum(g.count for g in shape.acc_groups)
    acc_def_at = np.zeros(n_acc, dtype=np.int64)
    acc_read_at = np.zeros(n_acc, dtype=np.int64)
    specials: List[List[Tuple[float, int, int]]] = [[] for _ in range(nB)]
    a0 = 0
    for g in shape.acc_groups:
        for a in range(g.count):
            specials[g.def_block].append(((a + 0.5) / g.count, KIND_ACC_DEF, a0 + a))
            specials[g.read_block].append(((a + 0.5) / g.count, KIND_ACC_READ, a0 + a))
        for ub in g.update_blocks:
            reps = max(1, int(np.floor(0.12 * sizes[ub] / g.count + 0.5)))
            for rep in range(reps):
                for a in range(g.count):
                    specials[ub].append(((rep * g.count + a + 0.5) / (reps * g.count), KIND_ACC_UPD, a0 + a))
        a0 += g.count
    for b in range(nB):
        sp = sorted(specials[b])
        if len(sp) >= sizes[b] and len(sp) > 0:
            raise ValueError(f"block {b} too small for its accumulator instructions")
        for k, (_, kd, acc) in enumerate(sp):
            i = int(blk_off[b] + ((2 * k + 1) * sizes[b]) // (2 * len(sp)))
            kind[i] = kd
            acc_of[i] = acc
            if kd == KIND_ACC_DEF:
                acc_def_at[acc] = i
            elif kd == KIND_ACC_READ:
                acc_read_at[acc] = i

    # ---- vreg pools: accumulators get ids [0, n_acc), then one pool per block
    pool_def = (kind == KIND_NORMAL) | (kind == KIND_ACC_READ)
    m_b = np.array([int(pool_def[blk_off[b]:blk_off[b + 1]].sum()) for b in range(nB)], dtype=np.int64)
    V = shape.n_vregs
    pool_size = _largest_remainder(V - n_acc, m_b, m_b)
    pool_base = n_acc + np.concatenate([[0], np.cumsum(pool_size)[:-1]])
    pool_n = np.zeros(nI, dtype=np.int64)       # pool-defining instructions before i in its block
    pool_pos: List[np.ndarray] = []
    def_vreg = np.zeros(nI, dtype=np.int64)
    for b in range(nB):
        sl = slice(int(blk_off[b]), int(blk_off[b + 1]))
        pd = pool_def[sl]
        before = np.cumsum(pd) - pd
        pool_n[sl] = before
        pool_pos.append(np.nonzero(pd)[0] + int(blk_off[b]))
        dv = np.where(pd, pool_base[b] + before % max(1, pool_size[b]), acc_of[sl])
        def_vreg[sl] = dv

    # ---- widths
    ws = np.array(sorted(shape.widths), dtype=np.int64)
    cum = np.cumsum([shape.widths[int(w)] for w in ws])
    cum = cum / cum[-1]
    width = ws[np.minimum(np.searchsorted(cum, rnd_unit(seed, _S_WIDTH, np.arange(V)), side="right"), len(ws) - 1)]
    if n_acc:
        aw = width[:n_acc]
        while aw.sum() > shape.P // 2 and aw.max() > 1:
            j = int(np.argmax(aw))
            aw[j] //= 2

    # ---- reads: forced accumulator read + geometric-recency picks
    u = np.searchsorted(np.array([0.1, 0.3, 0.6]), rnd_unit(seed, _S_UCOUNT, np.arange(nI)), side="right")
    nslot = np.where(kind == KIND_ACC_UPD, 2, np.where(kind == KIND_ACC_READ, np.maximum(u - 1, 0), u))
    slot_idx = np.arange(nI)[:, None] * 4 + np.arange(3)[None, :]
    G = np.floor(np.log1p(-rnd_unit(seed, _S_GEOM, slot_idx.ravel())) / np.log(0.7)).astype(np.int64).reshape(nI, 3)
    chains = _dominator_chains(nB, shape.edges)
    src = np.full((nI, 3), -1, dtype=np.int64)       # instruction whose value is read, -1 = dropped
    for b in range(nB):
        lo, hi = int(blk_off[b]), int(blk_off[b + 1])
        if hi == lo:
            continue
        n = pool_n[lo:hi][:, None]
        g = G[lo:hi].copy()
        active = np.arange(3)[None, :] < nslot[lo:hi][:, None]
        local_len = np.minimum(n, pool_size[b])
        res = np.full(g.shape, -1, dtype=np.int64)
        hit = active & (g < local_len)
        if hit.any():
            res[hit] = pool_pos[b][(n - 1 - g)[hit]]
        rem = active & ~hit
        g = g - local_len
        for d in chains[b]:
            ln = min(int(m_b[d]), int(pool_size[d]))
            hit = rem & (g < ln)
            if hit.any():
                res[hit] = pool_pos[d][(m_b[d] - 1 - g)[hit]]
            rem = rem & ~hit
            g = g - ln
        src[lo:hi] = res

    # ---- operand CSR: [def, forced acc read?, picks...]
    forced = (kind == KIND_ACC_UPD) | (kind == KIND_ACC_READ)
    n_ops = 1 + forced.astype(np.int64) + (src >= 0).sum(axis=1)
    op_off = np.concatenate([[0], np.cumsum(n_ops)]).astype(np.int64)
    nO = int(op_off[-1])
    op_vreg = np.zeros(nO, dtype=np.int64)
    op_vreg[op_off[:-1]] = def_vreg
    cur = op_off[:-1] + 1
    op_vreg[cur[forced]] = acc_of[forced]
    cur = cur + forced
    use_i, use_j = [], []
    for s in range(3):
        ok = src[:, s] >= 0
        op_vreg[cur[ok]] = def_vreg[src[ok, s]]
        use_i.append(np.nonzero(ok)[0])
        use_j.append(src[ok, s])
        cur = cur + ok
    use_i = np.concatenate(use_i)
    use_j = np.concatenate(use_j)

    # ---- CFG CSR
    succ_lists = [[] for _ in range(nB)]
    for a, b in shape.edges:
        succ_lists[a].append(b)
    succ_off = np.concatenate([[0], np.cumsum([len(s) for s in succ_lists])]).astype(np.uint32)
    succ = np.array([t for s in succ_lists for t in s], dtype=np.uint32)

    # ---- construction-time live intervals of every value (occupied = [def, last])
    ext = use_i.copy()
    bi, bj = blk_of[use_i], blk_of[use_j]
    for f, l in shape.loops:
        inside_i = (bi >= f) & (bi <= l)
        inside_j = (bj >= f) & (bj <= l)
        ext = np.where(inside_i & ~inside_j, np.maximum(ext, blk_off[l + 1]), ext)
    val_end = np.arange(nI)                       # exclusive end of "live after" points
    np.maximum.at(val_end, use_j, ext)
    val_last = np.maximum(np.arange(nI), val_end - 1)
    # accumulators: occupied from their definition to their last read, stretched the same way
    acc_last = np.zeros(n_acc, dtype=np.int64)
    if n_acc:
        fi = np.nonzero(forced)[0]
        fa = acc_of[fi]
        fext = fi.copy()
        fbi, fbj = blk_of[fi], blk_of[acc_def_at[fa]]
        for f, l in shape.loops:
            inside_i = (fbi >= f) & (fbi <= l)
            inside_j = (fbj >= f) & (fbj <= l)
            fext = np.where(inside_i & ~inside_j, np.maximum(fext, blk_off[l + 1]), fext)
        np.maximum.at(acc_last, fa, fext - 1)
    local = bi == bj
    last_local_use = np.arange(nI)
    np.maximum.at(last_local_use, use_j[local], use_i[local])

    prog = Program(
        n_blocks=nB, n_instrs=nI, n_vregs=V, n_operands=nO, n_edges=len(succ), P=shape.P, B=shape.B,
        block_instr_off=blk_off.astype(np.uint32), succ_off=succ_off, succ=succ,
        instr_op_off=op_off.astype(np.uint32), instr_n_defs=np.ones(nI, dtype=np.uint8),
        op_vreg=op_vreg.astype(np.uint32), vreg_width=width.astype(np.uint8),
    )
    prog.gen = dict(
        shape=shape, seed=seed, kind=kind, def_vreg=def_vreg, n_acc=n_acc,
        acc_def_at=acc_def_at, acc_read_at=acc_read_at, acc_last=acc_last, val_last=val_last,
        last_local_use=last_local_use, pool_def=pool_def, blk_of=blk_of,
    )
    return prog


# --------------------------------------------------------------- base allocation
def base_allocation(prog: Program) -> np.ndarray:
    """First-fit allocation (accumulators first, then vregs by first definition) with
    width-aligned bases over the construction-time occupancy of each vreg.  Two vregs
    that are ever occupied at the same instruction get disjoint register ranges."""
    g = prog.gen
    nI, V, P = prog.n_instrs, prog.n_vregs, prog.P
    width = prog.vreg_width.astype(np.int64)
    n_acc = g["n_acc"]
    base = np.full(V, -1, dtype=np.int64)
    occ = np.zeros((P, nI), dtype=bool)

    def first_fit(busy: np.ndarray, w: int) -> int:
        slots = P // w
        free = ~busy[: slots * w].reshape(slots, w).any(axis=1)
        idx = np.nonzero(free)[0]
        if len(idx) == 0:
            raise RuntimeError("register file too small for this program")
        return int(idx[0]) * w

    # accumulators: one interval each, definition to last read
    a_lo = g["acc_def_at"]
    a_hi = g["acc_last"]
    for a in range(n_acc):
        busy = np.zeros(P, dtype=bool)
        for c in range(a):
            if a_lo[c] <= a_hi[a] and a_lo[a] <= a_hi[c]:
                busy[base[c]: base[c] + width[c]] = True
        base[a] = first_fit(busy, int(width[a]))
    for a in range(n_acc):
        occ[base[a]: base[a] + width[a], a_lo[a]: a_hi[a] + 1] = True

    # pool vregs in order of first definition; one interval per defined value
    pool_instr = np.nonzero(g["pool_def"])[0]
    order = np.argsort(g["def_vreg"][pool_instr], kind="stable")
    pv = g["def_vreg"][pool_instr][order]
    pj = pool_instr[order]
    starts = np.nonzero(np.concatenate([[True], pv[1:] != pv[:-1]]))[0]
    ends = np.concatenate([starts[1:], [len(pv)]])
    first_def = pj[starts]
    val_last = g["val_last"]
    for gi in np.argsort(first_def, kind="stable"):
        v = int(pv[starts[gi]])
        js = pj[starts[gi]: ends[gi]]
        busy = np.zeros(P, dtype=bool)
        for j in js:
            busy |= occ[:, j: val_last[j] + 1].any(axis=1)
        b = first_fit(busy, int(width[v]))
        base[v] = b
        for j in js:
            occ[b: b + width[v], j: val_last[j] + 1] = True
    return base


def build_program(shape: Shape, seed: int, max_bumps: int = 16) -> Program:
    """Program plus a valid base allocation; bumps the seed when first-fit overflows P."""
    last = None
    for bump in range(max_bumps):
        prog = make_program(shape, seed + 1000003 * bump)
        try:
            prog.gen["base"] = base_allocation(prog)
            prog.gen["seed_bumps"] = bump
            _index_occurrences(prog)
            return prog
        except RuntimeError as e:      # register file too small: try the next seed
            last = e
    raise RuntimeError(f"no allocatable program for {shape.name} seed {seed}: {last}")


def _index_occurrences(prog: Program) -> None:
    g = prog.gen
    order = np.argsort(prog.op_vreg, kind="stable")
    counts = np.bincount(prog.op_vreg, minlength=prog.n_vregs)
    g["occ_off"] = np.concatenate([[0], np.cumsum(counts)])
    g["occ_idx"] = order
    first = np.zeros(prog.n_operands, dtype=bool)
    has = counts > 0
    first[order[g["occ_off"][:-1][has]]] = True
    g["non_first_ops"] = np.nonzero(~first)[0]
    g["op_instr"] = np.repeat(np.arange(prog.n_instrs), np.diff(prog.instr_op_off.astype(np.int64)))
    # lowest-index defining instruction of every vreg (operand 0 of an instruction is its def)
    fd = np.full(prog.n_vregs, prog.n_instrs, dtype=np.int64)
    np.minimum.at(fd, g["def_vreg"], np.arange(prog.n_instrs))
    g["first_def_instr"] = fd


# -------------------------------------------------------------------- candidates
def candidate_rows(prog: Program, K: int, fault_rate: float, seed: int,
                   k0: int = 0, k1: int | None = None, out: np.ndarray | None = None,
                   chunk: int = 128) -> Tuple[np.ndarray, np.ndarray]:
    """Rows k0..k1 of the K-row candidate matrix (uint16 [rows, pitch]) and a fault
    record per row: (kind, instr, vreg, other_vreg, operand), -1 where not applicable.

    Valid rows are a random validity-preserving renaming of the base allocation
    (permute the aligned groups of W = max width registers, xor the offset inside each
    group).  A faulted row carries exactly one fault: an inconsistent occurrence, a vreg
    moved onto the range of a value that is certainly live at one of its definitions, or
    a vreg moved out of the register file."""
    g = prog.gen
    if k1 is None:
        k1 = K
    n = k1 - k0
    pitch = prog.pitch
    if out is None:
        out = np.zeros((n, pitch), dtype=np.uint16)
    assert out.shape == (n, pitch) and out.dtype == np.uint16
    faults = np.full((n, 5), -1, dtype=np.int32)
    faults[:, 0] = FAULT_NONE
    base = g["base"]
    width = prog.vreg_width.astype(np.int64)
    P = prog.P
    W = int(width.max())
    assert P % W == 0 and (W & (W - 1)) == 0
    ng = P // W
    grp, off = base // W, base % W
    opv = prog.op_vreg.astype(np.int64)
    nO = prog.n_operands
    for c0 in range(k0, k1, chunk):
        c1 = min(k1, c0 + chunk)
        ks = np.arange(c0, c1)
        keys = rnd_u64(seed, _S_PERM, (ks[:, None] * ng + np.arange(ng)[None, :]).ravel()).reshape(len(ks), ng)
        perm = np.argsort(keys, axis=1, kind="stable")
        xo = (rnd_u64(seed, _S_XOR, (ks[:, None] * ng + np.arange(ng)[None, :]).ravel())
              .reshape(len(ks), ng) & U64(W - 1)).astype(np.int64)
        rows_idx = np.arange(len(ks))[:, None]
        tab = perm[rows_idx, grp[None, :]] * W + ((off[None, :] ^ xo[rows_idx, grp[None, :]]) & ~(width[None, :] - 1))
        tab = tab.astype(np.uint16)
        out[c0 - k0: c1 - k0, :nO] = tab[:, opv]
        out[c0 - k0: c1 - k0, nO:] = 0
        is_faulted = rnd_unit(seed, _S_FAULT, ks) < fault_rate
        for r in np.nonzero(is_faulted)[0]:
            _inject(prog, seed, int(ks[r]), out[c0 - k0 + r], tab[r], faults[c0 - k0 + r])
    return out, faults


# ---------------------------------------------------- dictionary form of a candidate
def dict_layout(prog: Program):
    """The per-basic-block dictionary form of a candidate row (the form the paper's model emits: one
    vreg -> register dictionary per basic block): one entry per (block, vreg occurring in the block),
    blocks in program order, a block's vregs in the order of their first occurrence in the block.
    Returns (dict_off u32 [n_blocks+1], dict_vreg u32 [n_entries], first_op i64 [n_entries]) where
    first_op is the operand column of the entry's first occurrence in its block.  Input format only:
    nothing of the check is computed here."""
    opv = prog.op_vreg.astype(np.int64)
    iop = prog.instr_op_off.astype(np.int64)
    offs, vregs, firsts = [0], [], []
    for b in range(prog.n_blocks):
        o0, o1 = int(iop[int(prog.block_instr_off[b])]), int(iop[int(prog.block_instr_off[b + 1])])
        seg = opv[o0:o1]
        _, idx = np.unique(seg, return_index=True)
        idx = np.sort(idx)
        vregs.append(seg[idx])
        firsts.append(idx + o0)
        offs.append(offs[-1] + len(idx))
    cat = (lambda xs, dt: np.concatenate(xs).astype(dt) if xs and sum(len(x) for x in xs) else np.zeros(0, dtype=dt))
    return np.asarray(offs, dtype=np.uint32), cat(vregs, np.uint32), cat(firsts, np.int64)


def dict_pitch(n_entries: int) -> int:
    """Row pitch of dictionary rows in elements: the entry count rounded up to 8 (16-byte rows)."""
    return max(8, (n_entries + 7) // 8 * 8)


def dict_rows(prog: Program, rows: np.ndarray, layout=None) -> np.ndarray:
    """Dictionary rows (uint16 [K, dict_pitch]) standing for per-occurrence rows: every entry takes
    the register its vreg has at its first occurrence in the block.  (A per-occurrence row that is
    inconsistent inside one block has no dictionary form; the entry then keeps the first value.)"""
    _, vregs, first_op = layout if layout is not None else dict_layout(prog)
    rows = np.atleast_2d(rows)
    out = np.zeros((rows.shape[0], dict_pitch(len(vregs))), dtype=np.uint16)
    out[:, : len(vregs)] = rows[:, first_op]
    return out


def _inject(prog: Program, seed: int, k: int, row: np.ndarray, tab: np.ndarray, rec: np.ndarray) -> None:
    g = prog.gen
    P = prog.P
    width = prog.vreg_width.astype(np.int64)
    occ_off, occ_idx = g["occ_off"], g["occ_idx"]
    r = [int(x) for x in rnd_u64(seed, _S_FPICK, k * 8 + np.arange(8))]
    fk = 1 + int(rnd_u64(seed, _S_FKIND, k)[0] % U64(3))
    if fk == FAULT_INCONSISTENT and (len(g["non_first_ops"]) == 0 or P < 2):
        fk = FAULT_RANGE
    if fk == FAULT_INCONSISTENT:
        o = int(g["non_first_ops"][r[0] % len(g["non_first_ops"])])
        row[o] = (int(row[o]) + 1 + r[1] % (P - 1)) % P
        rec[:] = (FAULT_INCONSISTENT, g["op_instr"][o], prog.op_vreg[o], -1, o)
        return
    if fk == FAULT_OVERLAP:
        nI = prog.n_instrs
        for t in range(64):
            i = (r[0] + t * 0x9E3779B1) % nI
            v = int(g["def_vreg"][i])
            lo = max(0, i - 48)
            js = np.arange(lo, i)
            loc = js[(g["last_local_use"][lo:i] > i) & g["pool_def"][lo:i]]
            loc = [int(g["def_vreg"][j]) for j in loc if g["def_vreg"][j] != v]
            accs = np.nonzero((g["acc_def_at"] <= i) & (i <= g["acc_read_at"] - 1))[0]
            accs = [int(a) for a in accs if a != v]
            pick_from = loc if (loc and (r[1] & 1 or not accs)) else accs
            if not pick_from:
                continue
            u = pick_from[r[2] % len(pick_from)]
            nb = int(tab[u]) + r[3] % int(width[u])
            nb = min(nb, P - int(width[v]))
            row[occ_idx[occ_off[v]: occ_off[v + 1]]] = nb
            rec[:] = (FAULT_OVERLAP, i, v, u, -1)
            return
        fk = FAULT_RANGE
    # out of the register file: every occurrence of one vreg gets a base >= P
    counts = np.diff(occ_off)
    v = r[4] % prog.n_vregs
    while counts[v] == 0 or g["first_def_instr"][v] >= prog.n_instrs:
        v = (v + 1) % prog.n_vregs
    row[occ_idx[occ_off[v]: occ_off[v + 1]]] = P + r[5] % 64
    rec[:] = (FAULT_RANGE, g["first_def_instr"][v], v, -1, -1)


# ----------------------------------------------------------------------- configs
_W2 = {1: 0.70, 2: 0.20, 4: 0.10}
_W3 = {1: 0.60, 2: 0.25, 4: 0.15}
_W5 = {1: 0.50, 2: 0.25, 4: 0.15, 8: 0.10}


def shape_tiny() -> Shape:
    return Shape("tiny", [64], [], [], [], n_vregs=24, widths={1: 1.0}, P=16)


def shape_gemm() -> Shape:
    return Shape("gemm", [200, 1600, 200], [(0, 1), (1, 1), (1, 2)], [(1, 1)],
                 [AccGroup(64, 0, (1,), 2)], n_vregs=600, widths=_W2, P=256)


def shape_attention() -> Shape:
    return Shape("attention", [400, 1200, 4800, 1200, 400],
                 [(0, 1), (1, 2), (2, 2), (2, 3), (3, 1), (3, 4)], [(1, 3), (2, 2)],
                 [AccGroup(128, 0, (2, 3), 4)], n_vregs=2500, widths=_W3, P=512)


def shape_batch_member(index: int, seed: int = 0) -> Shape:
    """One of the 256 programs of the batch workload; sizes drawn from (seed, index)."""
    r = rnd_u64(seed, _S_SHAPE, index * 4 + np.arange(4))
    nI = 1000 + int(r[0] % U64(3001))
    L = 1 + int(r[1] % U64(4))
    V = min(300 + int(r[2] % U64(901)), nI * 45 // 100)   # never more vregs than ~half the definitions
    pro = epi = max(80, nI // 10)
    body = (nI - pro - epi) // L
    sizes = [pro] + [body] * L + [nI - pro - body * L]
    edges = []
    for j in range(L + 1):
        edges.append((j, j + 1))
        if 1 <= j <= L:
            edges.append((j, j))
    loops = [(j, j) for j in range(1, L + 1)]
    accs = [AccGroup(32, j - 1, (j,), j + 1) for j in range(1, L + 1)]
    return Shape(f"batch{index}", sizes, edges, loops, accs, n_vregs=V, widths=_W2, P=256)


def shape_stress(n_instrs: int = 32000, n_vregs: int = 10000) -> Shape:
    pct = [2, 4, 6, 30, 30, 6, 4, 4, 4, 4, 4, 2]
    sizes = [n_instrs * p // 100 for p in pct]
    sizes[3] += n_instrs - sum(sizes)
    edges = [(0, 1), (1, 2), (2, 3), (3, 4), (4, 3), (4, 5), (5, 2), (5, 6), (6, 1), (6, 7),
             (7, 8), (7, 9), (8, 10), (9, 10), (10, 11)]
    loops = [(1, 6), (2, 5), (3, 4)]
    accs = [AccGroup(64, 0, (1, 6), 7), AccGroup(64, 1, (2, 5), 6), AccGroup(128, 2, (3, 4), 5)]
    return Shape("stress", sizes, edges, loops, accs, n_vregs=n_vregs, widths=_W5, P=512)


@dataclass
class Workload:
    name: str
    shapes: List[Shape]
    seeds: List[int]
    K: int
    fault_rate: float


def workload(index: int) -> Workload:
    """The five benchmark workloads, 0-based."""
    if index == 0:
        return Workload("tiny", [shape_tiny()], [0], 100, 0.30)
    if index == 1:
        return Workload("gemm", [shape_gemm()], [1], 100, 0.20)
    if index == 2:
        return Workload("attention", [shape_attention()], [2], 1000, 0.10)
    if index == 3:
        return Workload("batch", [shape_batch_member(i) for i in range(256)], list(range(256)), 100, 0.15)
    if index == 4:
        return Workload("stress", [shape_stress()], [4], 10000, 0.05)
    raise IndexError(index)
