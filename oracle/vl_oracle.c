/*
 * CPU oracle for the candidate-allocation check.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the plain, slow, single-threaded statement of what the CUDA
 * library must compute.  It shares no code, header, table or helper with the
 * CUDA path; only tests, the smoke check and the benchmark's CPU-baseline leg
 * may call it.  Nothing here is tuned.
 *
 * What is checked (paper, Section 1, correctness conditions (1) and (2);
 * Section 3.4, "Consistency", "Safety", "Realizability"; Section 2, register
 * tuples and the 4-bank register file; Section 4.5, a dataflow violation is a
 * write that clobbers a value still live later):
 *
 *   liveness   backward dataflow over the control-flow graph to the least
 *              fixed point, then a backward walk of every block giving the
 *              set of virtual registers live after each instruction;
 *   C          every occurrence of a virtual register carries the physical
 *              register of its first occurrence (the table T);
 *   R          at every definition of v: [T[v], T[v]+width(v)) lies in [0,P);
 *              optionally also: T[v] is a multiple of the vreg's alignment, the
 *              range lies inside the registers of the vreg's class and holds no
 *              reserved register;
 *   I          at every definition of v at instruction i: that range is
 *              disjoint from the range of every other virtual register that
 *              is live after i or also defined by i;
 *   bank tally per instruction, distinct source base registers that share a
 *              bank (T mod B) cost one extra cycle each beyond the first.
 *
 * The paper states the properties, not an encoding; equivalence with the
 * authors' SMT verifier is therefore: parity unpinned.  Every function below
 * is pinned by the tests under tests/ against brute-force path enumeration,
 * closed forms and hand-worked programs.
 *
 * Conventions: an instruction's operands are its definitions followed by its
 * reads; operand index == column of the candidate row; reads happen before
 * writes inside one instruction.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    uint32_t n_blocks, n_instrs, n_vregs, n_operands, n_edges, P, B;
    const uint32_t *block_instr_off; /* [n_blocks+1] */
    const uint32_t *succ_off;        /* [n_blocks+1] */
    const uint32_t *succ;            /* [n_edges]    */
    const uint32_t *instr_op_off;    /* [n_instrs+1] */
    const uint8_t *instr_n_defs;     /* [n_instrs]   */
    const uint32_t *op_vreg;         /* [n_operands] */
    const uint8_t *vreg_width;       /* [n_vregs]    */
    /* Optional hardware constraints (Section 1: register file sizes and reserved registers;
     * Section 3.2: scalar / vector register classes; Section 4.5: hardware rules on register
     * tuples).  A null pointer switches the constraint off. */
    const uint8_t *vreg_align;       /* [n_vregs] the base register is a multiple of this (>= 1) */
    const uint8_t *vreg_class;       /* [n_vregs] register class of the vreg */
    const uint32_t *class_lo;        /* [classes] class c owns the registers [class_lo[c], class_hi[c]) */
    const uint32_t *class_hi;
    const uint8_t *reserved;         /* [P] 1 = no vreg may occupy this register */
} vlo_program;

typedef struct {
    uint32_t flags;                /* bit0 pass, bit1 inconsistent, bit2 out of range, bit3 interference */
    int32_t first_violation_instr; /* lowest instruction index with any violation, -1 if none */
    uint32_t conflict_pairs;       /* number of (instruction, definition, other vreg) overlaps */
    uint32_t bank_conflicts;       /* extra read cycles summed over instructions */
} vlo_verdict;

enum { VLO_PASS = 1, VLO_INCONSISTENT = 2, VLO_OUT_OF_RANGE = 4, VLO_INTERFERENCE = 8 };

/* ---------------------------------------------------------------- liveness */

/*
 * Block-level sets and fixed point (one byte per (block, vreg)).
 *   use[b] = vregs read in b before any write to them in b
 *   def[b] = vregs written in b
 *   out[b] = union of in[s] over successors s;  in[b] = use[b] | (out[b] - def[b])
 * starting from empty sets, sweeping until a sweep changes nothing.
 * order = 0 sweeps blocks last to first, order = 1 first to last; the least
 * fixed point does not depend on it.  Returns the number of sweeps.
 */
uint32_t vlo_block_liveness(const vlo_program *p, uint8_t *live_in, uint8_t *live_out, int order)
{
    const uint32_t nB = p->n_blocks, V = p->n_vregs;
    uint8_t *use = calloc((size_t)nB * V + 1, 1);
    uint8_t *def = calloc((size_t)nB * V + 1, 1);
    for (uint32_t b = 0; b < nB; ++b) {
        for (uint32_t i = p->block_instr_off[b]; i < p->block_instr_off[b + 1]; ++i) {
            uint32_t o0 = p->instr_op_off[i], o1 = p->instr_op_off[i + 1], nd = p->instr_n_defs[i];
            for (uint32_t o = o0 + nd; o < o1; ++o) { /* reads first */
                uint32_t v = p->op_vreg[o];
                if (!def[(size_t)b * V + v]) use[(size_t)b * V + v] = 1;
            }
            for (uint32_t o = o0; o < o0 + nd; ++o) def[(size_t)b * V + p->op_vreg[o]] = 1;
        }
    }
    memset(live_in, 0, (size_t)nB * V);
    memset(live_out, 0, (size_t)nB * V);
    uint32_t sweeps = 0;
    int changed = 1;
    while (changed) {
        changed = 0;
        ++sweeps;
        for (uint32_t n = 0; n < nB; ++n) {
            uint32_t b = order ? n : nB - 1 - n;
            for (uint32_t v = 0; v < V; ++v) {
                uint8_t o = 0;
                for (uint32_t e = p->succ_off[b]; e < p->succ_off[b + 1]; ++e)
                    o |= live_in[(size_t)p->succ[e] * V + v];
                uint8_t in = use[(size_t)b * V + v] | (o & !def[(size_t)b * V + v]);
                if (o != live_out[(size_t)b * V + v] || in != live_in[(size_t)b * V + v]) changed = 1;
                live_out[(size_t)b * V + v] = o;
                live_in[(size_t)b * V + v] = in;
            }
        }
    }
    free(use);
    free(def);
    return sweeps;
}

/*
 * Per-instruction live-after sets in CSR form, ascending vreg id.
 * Walk each block backwards from out[b]:  live_after(i) = live;
 * live = (live - defs(i)) | reads(i).
 * lo_off has n_instrs+1 entries.  At most cap ids are stored in lo; the total
 * count is returned (call once with cap = 0 to size the buffer).
 */
uint64_t vlo_instr_liveness(const vlo_program *p, const uint8_t *blk_live_out,
                            uint64_t *lo_off, uint32_t *lo, uint64_t cap)
{
    const uint32_t V = p->n_vregs, nI = p->n_instrs;
    uint8_t *live = malloc((size_t)V + 1);
    uint64_t *cnt = calloc((size_t)nI + 1, sizeof(uint64_t));
    /* pass 1: sizes */
    for (uint32_t b = 0; b < p->n_blocks; ++b) {
        memcpy(live, blk_live_out + (size_t)b * V, V);
        for (uint32_t i = p->block_instr_off[b + 1]; i-- > p->block_instr_off[b];) {
            uint64_t c = 0;
            for (uint32_t v = 0; v < V; ++v) c += live[v];
            cnt[i] = c;
            uint32_t o0 = p->instr_op_off[i], o1 = p->instr_op_off[i + 1], nd = p->instr_n_defs[i];
            for (uint32_t o = o0; o < o0 + nd; ++o) live[p->op_vreg[o]] = 0;
            for (uint32_t o = o0 + nd; o < o1; ++o) live[p->op_vreg[o]] = 1;
        }
    }
    uint64_t total = 0;
    for (uint32_t i = 0; i < nI; ++i) { lo_off[i] = total; total += cnt[i]; }
    lo_off[nI] = total;
    /* pass 2: ids */
    for (uint32_t b = 0; b < p->n_blocks; ++b) {
        memcpy(live, blk_live_out + (size_t)b * V, V);
        for (uint32_t i = p->block_instr_off[b + 1]; i-- > p->block_instr_off[b];) {
            uint64_t at = lo_off[i];
            for (uint32_t v = 0; v < V; ++v)
                if (live[v]) { if (at < cap) lo[at] = v; ++at; }
            uint32_t o0 = p->instr_op_off[i], o1 = p->instr_op_off[i + 1], nd = p->instr_n_defs[i];
            for (uint32_t o = o0; o < o0 + nd; ++o) live[p->op_vreg[o]] = 0;
            for (uint32_t o = o0 + nd; o < o1; ++o) live[p->op_vreg[o]] = 1;
        }
    }
    free(live);
    free(cnt);
    return total;
}

/* ------------------------------------------------------------------ verify */

static int ranges_overlap(uint32_t a, uint32_t wa, uint32_t b, uint32_t wb)
{
    return a < b + wb && b < a + wa; /* plain integers, no wrap: a,b <= 65535, w <= 255 */
}

/*
 * Core walk shared by the three reporting functions below (they differ only in
 * what they write down).  kinds, if given, receives per instruction the OR of
 * the violation bits raised there; triples, if given, receives up to cap
 * (instruction, defined vreg, other vreg) overlap records; *n_triples counts all.
 */
static void walk(const vlo_program *p, const uint64_t *lo_off, const uint32_t *lo,
                 const uint16_t *row, vlo_verdict *out, uint8_t *kinds,
                 uint32_t *triples, uint64_t cap, uint64_t *n_triples, uint64_t *bank_hist)
{
    const uint32_t V = p->n_vregs, nI = p->n_instrs;
    int32_t *T = malloc(((size_t)V + 1) * sizeof(int32_t));
    for (uint32_t v = 0; v < V; ++v) T[v] = -1;
    uint32_t *Q = malloc(((size_t)p->n_operands + 1) * sizeof(uint32_t));
    uint32_t flags = 0, pairs = 0, bank = 0;
    int64_t first = -1;
    uint64_t nt = 0;
    if (kinds) memset(kinds, 0, nI);

    /* table and consistency: operands in program order, first occurrence wins */
    for (uint32_t i = 0; i < nI; ++i) {
        for (uint32_t o = p->instr_op_off[i]; o < p->instr_op_off[i + 1]; ++o) {
            uint32_t v = p->op_vreg[o];
            if (T[v] < 0) T[v] = row[o];
            else if ((uint32_t)T[v] != row[o]) {
                flags |= VLO_INCONSISTENT;
                if (kinds) kinds[i] |= VLO_INCONSISTENT;
                if (first < 0 || (int64_t)i < first) first = i;
            }
        }
    }

    for (uint32_t i = 0; i < nI; ++i) {
        uint32_t o0 = p->instr_op_off[i], o1 = p->instr_op_off[i + 1], nd = p->instr_n_defs[i];
        for (uint32_t d = o0; d < o0 + nd; ++d) {
            uint32_t v = p->op_vreg[d];
            uint32_t s = (uint32_t)T[v], w = p->vreg_width[v];
            int bad = 0;
            /* realizability: the tuple fits in the register file and keeps the hardware rules */
            int unreal = s + w > p->P;
            if (p->vreg_align && s % p->vreg_align[v] != 0) unreal = 1;
            if (p->vreg_class) {
                uint32_t c = p->vreg_class[v];
                if (s < p->class_lo[c] || s + w > p->class_hi[c]) unreal = 1;
            }
            if (p->reserved)
                for (uint32_t r = s; r < s + w && r < p->P; ++r)
                    if (p->reserved[r]) unreal = 1;
            if (unreal) {
                flags |= VLO_OUT_OF_RANGE;
                if (kinds) kinds[i] |= VLO_OUT_OF_RANGE;
                bad = 1;
            }
            /* safety: every other vreg live after i ... */
            for (uint64_t e = lo_off[i]; e < lo_off[i + 1]; ++e) {
                uint32_t u = lo[e];
                if (u == v) continue;
                if (ranges_overlap(s, w, (uint32_t)T[u], p->vreg_width[u])) {
                    ++pairs;
                    if (triples && nt < cap) { triples[3 * nt] = i; triples[3 * nt + 1] = v; triples[3 * nt + 2] = u; }
                    ++nt;
                    flags |= VLO_INTERFERENCE;
                    if (kinds) kinds[i] |= VLO_INTERFERENCE;
                    bad = 1;
                }
            }
            /* ... and every other vreg written by the same instruction that is not live after it */
            for (uint32_t d2 = o0; d2 < o0 + nd; ++d2) {
                uint32_t u = p->op_vreg[d2];
                if (u == v) continue;
                int in_live = 0;
                for (uint64_t e = lo_off[i]; e < lo_off[i + 1]; ++e) if (lo[e] == u) in_live = 1;
                if (in_live) continue;
                if (ranges_overlap(s, w, (uint32_t)T[u], p->vreg_width[u])) {
                    ++pairs;
                    if (triples && nt < cap) { triples[3 * nt] = i; triples[3 * nt + 1] = v; triples[3 * nt + 2] = u; }
                    ++nt;
                    flags |= VLO_INTERFERENCE;
                    if (kinds) kinds[i] |= VLO_INTERFERENCE;
                    bad = 1;
                }
            }
            if (bad && (first < 0 || (int64_t)i < first)) first = i;
        }
        /* bank tally: Q = distinct source base registers of this instruction; every
         * bank holding n of them costs n-1 extra cycles */
        uint32_t nq = 0;
        for (uint32_t a = o0 + nd; a < o1; ++a) {
            uint32_t ta = (uint32_t)T[p->op_vreg[a]];
            int dup = 0;
            for (uint32_t q = 0; q < nq; ++q) if (Q[q] == ta) dup = 1;
            if (!dup) Q[nq++] = ta;
        }
        for (uint32_t q = 0; q < nq; ++q) {
            int first_of_bank = 1;
            for (uint32_t r = 0; r < q; ++r) if (Q[r] % p->B == Q[q] % p->B) first_of_bank = 0;
            if (!first_of_bank) continue;
            uint32_t n = 0;
            for (uint32_t r = 0; r < nq; ++r) if (Q[r] % p->B == Q[q] % p->B) ++n;
            bank += n - 1;
            if (bank_hist) bank_hist[Q[q] % p->B] += n - 1;
        }
    }
    free(Q);
    if (!flags) flags = VLO_PASS;
    out->flags = flags;
    out->first_violation_instr = (int32_t)first;
    out->conflict_pairs = pairs;
    out->bank_conflicts = bank;
    if (n_triples) *n_triples = nt;
    free(T);
}

void vlo_verify(const vlo_program *p, const uint64_t *lo_off, const uint32_t *lo,
                const uint16_t *row, vlo_verdict *out)
{
    walk(p, lo_off, lo, row, out, NULL, NULL, 0, NULL, NULL);
}

void vlo_verify_rows(const vlo_program *p, const uint64_t *lo_off, const uint32_t *lo,
                     const uint16_t *rows, uint64_t K, uint64_t pitch, vlo_verdict *out)
{
    for (uint64_t k = 0; k < K; ++k) walk(p, lo_off, lo, rows + k * pitch, out + k, NULL, NULL, 0, NULL, NULL);
}

/* per-instruction violation kinds for one row */
void vlo_violations(const vlo_program *p, const uint64_t *lo_off, const uint32_t *lo,
                    const uint16_t *row, uint8_t *kinds)
{
    vlo_verdict v;
    walk(p, lo_off, lo, row, &v, kinds, NULL, 0, NULL, NULL);
}

/* every (instruction, defined vreg, other vreg) overlap of one row; returns the total */
uint64_t vlo_conflicts(const vlo_program *p, const uint64_t *lo_off, const uint32_t *lo,
                       const uint16_t *row, uint32_t *triples, uint64_t cap)
{
    vlo_verdict v;
    uint64_t n = 0;
    walk(p, lo_off, lo, row, &v, NULL, triples, cap, &n, NULL);
    return n;
}

/* extra read cycles of one row per register bank: hist[b] sums, over the instructions, the
 * distinct source registers in bank b beyond the first (hist must hold B zeroed counters) */
void vlo_bank_histogram(const vlo_program *p, const uint64_t *lo_off, const uint32_t *lo,
                        const uint16_t *row, uint64_t *hist)
{
    vlo_verdict v;
    for (uint32_t b = 0; b < p->B; ++b) hist[b] = 0;
    walk(p, lo_off, lo, row, &v, NULL, NULL, 0, NULL, hist);
}

/*
 * Registers the definitions of instruction i must keep off (Section 4.5 proposes decoding that masks
 * out the registers occupied at that point): occ[i * P + r] = 1 iff register r < P belongs to the
 * range of a vreg that is live after i and not defined by i, or is reserved.  A vreg whose table
 * entry is P or more (not assigned yet) contributes nothing.
 */
void vlo_occupied(const vlo_program *p, const uint64_t *lo_off, const uint32_t *lo,
                  const uint16_t *row, uint8_t *occ)
{
    const uint32_t V = p->n_vregs, nI = p->n_instrs, P = p->P;
    int32_t *T = malloc(((size_t)V + 1) * sizeof(int32_t));
    for (uint32_t v = 0; v < V; ++v) T[v] = -1;
    for (uint32_t o = 0; o < p->n_operands; ++o)
        if (T[p->op_vreg[o]] < 0) T[p->op_vreg[o]] = row[o];
    memset(occ, 0, (size_t)nI * P);
    for (uint32_t i = 0; i < nI; ++i) {
        uint32_t o0 = p->instr_op_off[i], nd = p->instr_n_defs[i];
        for (uint64_t e = lo_off[i]; e < lo_off[i + 1]; ++e) {
            uint32_t u = lo[e];
            int own = 0;
            for (uint32_t d = o0; d < o0 + nd; ++d) if (p->op_vreg[d] == u) own = 1;
            if (own) continue;
            for (uint32_t r = (uint32_t)T[u]; r < (uint32_t)T[u] + p->vreg_width[u]; ++r)
                if (r < P) occ[(size_t)i * P + r] = 1;
        }
        if (p->reserved)
            for (uint32_t r = 0; r < P; ++r) if (p->reserved[r]) occ[(size_t)i * P + r] = 1;
    }
    free(T);
}

/* ------------------------------------------------- dictionary candidates */

/*
 * The model of the paper does not emit one register per operand occurrence: it emits, for every
 * basic block, a dictionary from the block's virtual registers to physical registers (Section 3.1:
 * the assignment is generated "per basic block" along the control-flow graph, as a JSON-style
 * dictionary; Section 3.2: registers are renumbered per block, so the same virtual register shows
 * up in the dictionaries of several blocks).  A candidate in that form is one 16-bit value per
 * (block, virtual register occurring in the block).
 *
 * Layout of such a row (a reading: the paper fixes no order inside a dictionary): blocks in program
 * order; inside a block its virtual registers in the order of their first occurrence in the block
 * (definitions of an instruction before its reads).  vlo_dict_layout writes dict_off[n_blocks+1],
 * and, per entry, the vreg and the first instruction of the block in which it occurs; it returns the
 * number of entries (the arrays must hold n_operands entries at most).
 *
 * Meaning: every occurrence of v inside block b carries the register of entry (b, v).  The check is
 * then the check of that per-occurrence assignment: Consistency compares the entries of one vreg
 * across blocks (the entry of the lowest block that uses it is the table value; a differing entry is
 * a violation reported at the first instruction of its block that touches the vreg), everything
 * else follows from the table as before.
 */
uint32_t vlo_dict_layout(const vlo_program *p, uint32_t *dict_off, uint32_t *dict_vreg, uint32_t *entry_instr)
{
    uint32_t n = 0;
    uint8_t *seen = malloc((size_t)p->n_vregs + 1);
    for (uint32_t b = 0; b < p->n_blocks; ++b) {
        dict_off[b] = n;
        memset(seen, 0, (size_t)p->n_vregs + 1);
        for (uint32_t i = p->block_instr_off[b]; i < p->block_instr_off[b + 1]; ++i)
            for (uint32_t o = p->instr_op_off[i]; o < p->instr_op_off[i + 1]; ++o) {
                uint32_t v = p->op_vreg[o];
                if (seen[v]) continue;
                seen[v] = 1;
                dict_vreg[n] = v;
                entry_instr[n] = i;
                ++n;
            }
    }
    dict_off[p->n_blocks] = n;
    free(seen);
    return n;
}

/* rows of dictionary candidates, pitch entries apart, checked one by one */
void vlo_verify_dict_rows(const vlo_program *p, const uint64_t *lo_off, const uint32_t *lo,
                          const uint16_t *rows, uint64_t K, uint64_t pitch, vlo_verdict *out)
{
    uint32_t *dict_off = malloc(((size_t)p->n_blocks + 1) * sizeof(uint32_t));
    uint32_t *dict_vreg = malloc(((size_t)p->n_operands + 1) * sizeof(uint32_t));
    uint32_t *entry_instr = malloc(((size_t)p->n_operands + 1) * sizeof(uint32_t));
    uint16_t *occ = malloc(((size_t)p->n_operands + 1) * sizeof(uint16_t));
    uint32_t *entry_of = malloc(((size_t)p->n_vregs + 1) * sizeof(uint32_t));
    vlo_dict_layout(p, dict_off, dict_vreg, entry_instr);
    for (uint64_t k = 0; k < K; ++k) {
        const uint16_t *row = rows + k * pitch;
        /* the per-occurrence assignment the dictionaries stand for */
        for (uint32_t b = 0; b < p->n_blocks; ++b) {
            for (uint32_t e = dict_off[b]; e < dict_off[b + 1]; ++e) entry_of[dict_vreg[e]] = e;
            for (uint32_t i = p->block_instr_off[b]; i < p->block_instr_off[b + 1]; ++i)
                for (uint32_t o = p->instr_op_off[i]; o < p->instr_op_off[i + 1]; ++o)
                    occ[o] = row[entry_of[p->op_vreg[o]]];
        }
        walk(p, lo_off, lo, occ, out + k, NULL, NULL, 0, NULL, NULL);
    }
    free(entry_of); free(occ); free(entry_instr); free(dict_vreg); free(dict_off);
}

/* ------------------------------------------------- re-sampling statistics */

/*
 * The verifier sits in a loop that samples the model again until a candidate
 * passes or the attempts run out (paper, Section 3.4, last paragraph).  The
 * figures the paper reports about that loop (Section 4, before "Main
 * Results"): Pass@k, the share of test cases with a passing candidate among
 * their first k attempts; AvgTry and MaxTry, the average and the largest
 * number of attempts up to and including the first passing one, over the test
 * cases that reached one.  Rows are attempts, in order.
 */
typedef struct {
    uint64_t first_pass; /* row of the first passing verdict, K if there is none */
    uint64_t n_pass;     /* passing verdicts among the K rows */
} vlo_sample_stats;

void vlo_sample_stats_of(const vlo_verdict *out, uint64_t K, vlo_sample_stats *s)
{
    s->first_pass = K;
    s->n_pass = 0;
    for (uint64_t k = 0; k < K; ++k) {
        if (!(out[k].flags & VLO_PASS)) continue;
        if (s->first_pass == K) s->first_pass = k;
        s->n_pass += 1;
    }
}

/*
 * summary[0] = test cases, [1] = solved ones, [2] = sum of attempts over the
 * solved ones, [3] = largest number of attempts of a solved one (0 if none),
 * [4 + j] = test cases solved within their first k[j] attempts.
 */
void vlo_resample_summary(uint32_t n, const vlo_sample_stats *s, const uint64_t *K,
                          uint32_t n_k, const uint32_t *k, uint64_t *summary)
{
    for (uint32_t j = 0; j < 4 + n_k; ++j) summary[j] = 0;
    summary[0] = n;
    for (uint32_t c = 0; c < n; ++c) {
        if (s[c].first_pass >= K[c]) continue; /* never passed */
        const uint64_t attempts = s[c].first_pass + 1;
        summary[1] += 1;
        summary[2] += attempts;
        if (attempts > summary[3]) summary[3] = attempts;
        for (uint32_t j = 0; j < n_k; ++j)
            if (attempts <= k[j]) summary[4 + j] += 1;
    }
}
