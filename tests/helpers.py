"""Test-side helpers: random small programs and brute-force definitions.

Everything here is written independently of both the oracle and the CUDA path:
liveness by explicit path search, interference by the all-pairs definition.
"""
from __future__ import annotations

import random
from typing import List, Set, Tuple

import numpy as np

from paper_2506_17506_b200 import synth


def random_program(seed: int, strict: bool = True, reachable: bool = True,
                   max_blocks: int = 6, max_instrs: int = 40, max_vregs: int = 12,
                   P: int = 16, widths=(1, 1, 1, 2, 2, 4), B: int = 4,
                   multi_def: bool = True) -> synth.Program:
    """Random CFG (loops, diamonds, self-edges, optionally unreachable blocks) with
    0..2 definitions and 0..4 reads per instruction.  With strict=True the entry block
    first defines every vreg, so nothing is live into the program."""
    rng = random.Random(seed)
    nB = rng.randint(1, max_blocks)
    V = rng.randint(2, max_vregs)
    blocks: List[List[Tuple[List[int], List[int]]]] = [[] for _ in range(nB)]
    if strict:
        vs = list(range(V))
        rng.shuffle(vs)
        while vs:
            n = 2 if (multi_def and len(vs) >= 2 and rng.random() < 0.3) else 1
            defs, vs = vs[:n], vs[n:]
            blocks[0].append((defs, []))
    budget = rng.randint(nB, max_instrs)
    for _ in range(budget):
        b = rng.randrange(nB)
        nd = rng.choice([0, 1, 1, 1, 1, 2] if multi_def else [0, 1, 1, 1])
        defs = rng.sample(range(V), min(nd, V))
        uses = [rng.randrange(V) for _ in range(rng.choice([0, 1, 2, 2, 3, 4]))]
        blocks[b].append((defs, uses))
    edges = set()
    if reachable:
        for b in range(nB - 1):
            edges.add((b, b + 1))
    for _ in range(rng.randint(0, 2 * nB)):
        a, b = rng.randrange(nB), rng.randrange(nB)
        if reachable or a != 0 or rng.random() < 0.5:
            edges.add((a, b))
    ws = [rng.choice(widths) for _ in range(V)]
    return synth.program_from_lists(blocks, sorted(edges), V, ws, P, B)


def instr_lists(p: synth.Program):
    """[(defs, uses)] per instruction, block id per instruction, successor lists."""
    ins = []
    for i in range(p.n_instrs):
        o0, o1, nd = int(p.instr_op_off[i]), int(p.instr_op_off[i + 1]), int(p.instr_n_defs[i])
        ops = [int(x) for x in p.op_vreg[o0:o1]]
        ins.append((ops[:nd], ops[nd:]))
    blk = np.repeat(np.arange(p.n_blocks), np.diff(p.block_instr_off.astype(np.int64)))
    succ = [[int(s) for s in p.succ[int(p.succ_off[b]): int(p.succ_off[b + 1])]] for b in range(p.n_blocks)]
    return ins, blk, succ


def path_liveness(p: synth.Program):
    """live_after[i] and block live_in / live_out by the path definition:
    v is live at a point iff some CFG path from it reaches a read of v before any
    write of v (reads of an instruction come before its writes)."""
    ins, blk, succ = instr_lists(p)
    boff = [int(x) for x in p.block_instr_off]

    def live_from_block_entry(b0: int, v: int, seen_blocks: Set[int]) -> bool:
        # explicit stack of blocks entered from their first instruction
        stack = [b0]
        while stack:
            b = stack.pop()
            if b in seen_blocks:
                continue
            seen_blocks.add(b)
            killed = False
            for i in range(boff[b], boff[b + 1]):
                d, u = ins[i]
                if v in u:
                    return True
                if v in d:
                    killed = True
                    break
            if not killed:
                stack.extend(succ[b])
        return False

    def live_after_instr(i: int, v: int) -> bool:
        b = int(blk[i])
        for j in range(i + 1, boff[b + 1]):
            d, u = ins[j]
            if v in u:
                return True
            if v in d:
                return False
        seen: Set[int] = set()
        return any(live_from_block_entry(s, v, seen) for s in succ[b])

    V = p.n_vregs
    live_after = [[v for v in range(V) if live_after_instr(i, v)] for i in range(p.n_instrs)]
    blk_in = np.zeros((p.n_blocks, V), dtype=np.uint8)
    blk_out = np.zeros((p.n_blocks, V), dtype=np.uint8)
    for b in range(p.n_blocks):
        for v in range(V):
            blk_in[b, v] = live_from_block_entry(b, v, set())
            seen: Set[int] = set()
            blk_out[b, v] = any(live_from_block_entry(s, v, seen) for s in succ[b])
    return live_after, blk_in, blk_out


def table_of(p: synth.Program, row) -> dict:
    T = {}
    for o in range(p.n_operands):
        T.setdefault(int(p.op_vreg[o]), int(row[o]))
    return T


def overlap(a, wa, b, wb) -> bool:
    return a < b + wb and b < a + wa


def copointed_overlapping_pairs(p: synth.Program, live_after, row) -> Set[Tuple[int, int]]:
    """All-pairs definition: unordered vreg pairs that are together in
    live_after(i) | defs(i) for some i and whose register ranges intersect."""
    ins, _, _ = instr_lists(p)
    T = table_of(p, row)
    w = [int(x) for x in p.vreg_width]
    pairs = set()
    for i, (d, _) in enumerate(ins):
        here = sorted(set(live_after[i]) | set(d))
        for a in range(len(here)):
            for b in range(a + 1, len(here)):
                x, y = here[a], here[b]
                if overlap(T[x], w[x], T[y], w[y]):
                    pairs.add((x, y))
    return pairs


def row_from_table(p: synth.Program, T) -> np.ndarray:
    row = np.zeros(p.pitch, dtype=np.uint16)
    row[: p.n_operands] = np.asarray(T, dtype=np.int64)[p.op_vreg.astype(np.int64)]
    return row
