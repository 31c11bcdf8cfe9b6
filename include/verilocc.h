/*
 * verilocc.h -- C ABI of the batch verifier for register-allocation candidates.
 *
 * The library checks K candidate allocations of one program (a GPU kernel in
 * machine-IR form: basic blocks, CFG edges, per-instruction definitions and
 * reads of virtual registers, register-tuple widths) against the correctness
 * conditions of the paper:
 *   Section 1, conditions (1) and (2); Section 3.4 "Consistency", "Safety",
 *   "Realizability"; Section 2 (a wide value takes consecutive registers; the
 *   register file has 4 banks and reads from one bank stall).
 * The check is the polynomial-time one the paper names in Section 4.6 (following
 * control and data dependence), not an SMT query.
 *
 * All functions return VL_OK (0) or a negative VL_ERR_* code; none throws,
 * aborts or prints.  An invalid candidate is never an error, it is a verdict.
 * The library is not thread-safe per program handle; distinct handles may be
 * used from distinct threads.  There is no CPU fallback: every entry point that
 * computes needs a CUDA device of compute capability 10.0.
 */
#ifndef VERILOCC_H
#define VERILOCC_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    VL_OK = 0,
    VL_ERR_INVALID_ARG = -1,       /* null pointer, bad size, misaligned buffer */
    VL_ERR_MALFORMED_PROGRAM = -2, /* CSR offsets not monotone, ids out of range, zero width, duplicate def */
    VL_ERR_NOT_STRICT = -3,        /* some vreg is live into the entry block (read before any write) */
    VL_ERR_LIVENESS_NOT_RUN = -4,  /* vl_verify* before a successful vl_liveness */
    VL_ERR_UNSUPPORTED = -5,       /* program exceeds the shared-memory plan or a 32-bit size */
    VL_ERR_NO_CONVERGE = -6,       /* liveness did not reach its fixed point within n_blocks + 2 sweeps */
    VL_ERR_CUDA = -7,              /* a CUDA call failed; vl_last_cuda_error() has the code */
    VL_ERR_DEVICE_WAIT = -8        /* a bounded wait inside a kernel gave up (copy engine never signalled) */
};

/* Verdict flag bits.  VL_PASS is set iff none of the others is. */
enum { VL_PASS = 1u, VL_INCONSISTENT = 2u, VL_OUT_OF_RANGE = 4u, VL_INTERFERENCE = 8u };

/* Tunables for vl_program_set_option (set before vl_liveness). */
enum {
    VL_OPT_CHUNK_INSTRS = 1, /* instructions per walk chunk (default 160; long blocks get a chunk count that is a multiple of 8) */
    VL_OPT_GROUP = 2,        /* candidates per thread block of the table kernel: 0 = choose, else 1, 2, 4 or 8 */
    VL_OPT_THREADS = 3,      /* threads per thread block of the table kernel: 0 = choose, else 256 or 512 */
    VL_OPT_SUB_BATCH = 4,    /* candidates per pass of the verify kernels (multiple of 32, default 5120) */
    VL_OPT_KERNEL_TIMING = 5,/* 1: vl_verify records CUDA events around its kernels (see vl_kernel_times); may be
                                set at any time; setting it discards the events recorded so far */
    VL_OPT_LANES = 6,        /* internal streams the passes of vl_verify are spread over, 1..8 (default 3);
                                1 = every kernel in order on the caller's stream.  vl_verify_batch reads the
                                option of its first program: 1 = in order, anything else = all 8 streams */
    VL_OPT_PREFETCH_TILES = 8, /* tiles of the candidate rows that the table kernel (8 candidates per block) asks into
                                L2 ahead of its copy ring, 0..64 (default 3; 0 = none) */
    VL_OPT_STAGGER_US = 9,     /* the first wave of thread blocks of a call's first table kernel starts in four classes this
                                many microseconds apart (0..200, default 12), so that not all of them stream, then all of them
                                sweep, in step; only for calls of at least two waves */
    VL_OPT_TEST_WAIT = 7     /* test hook for the bounded device waits: 1 = the table kernel (8 candidates per
                                block) waits for its first tile on a barrier that nothing completes, with a short
                                poll limit, so that the wait runs out: the call still returns, its verdicts are
                                garbage and vl_verify_status reports VL_ERR_DEVICE_WAIT.  0 = normal (default) */
};

/*
 * Program descriptor.  All pointers are HOST memory, read during
 * vl_program_create only (borrowed, never freed, may be released afterwards).
 *
 * Instructions are numbered in layout order; block b owns instructions
 * [block_instr_off[b], block_instr_off[b+1]); block 0 is the entry.  The
 * operands of instruction i are [instr_op_off[i], instr_op_off[i+1]): first its
 * instr_n_defs[i] definitions, then its reads.  An operand's index is its
 * column in a candidate row.  Reads of an instruction happen before its writes.
 * A vreg of width w mapped to physical register p occupies [p, p+w).
 */
typedef struct {
    uint32_t n_blocks, n_instrs, n_vregs, n_operands, n_edges;
    uint32_t P;                      /* physical registers, 1..65535 */
    uint32_t B;                      /* register banks, >= 1 (bank = register mod B) */
    const uint32_t *block_instr_off; /* [n_blocks+1] */
    const uint32_t *succ_off;        /* [n_blocks+1] */
    const uint32_t *succ;            /* [n_edges] successor block ids */
    const uint32_t *instr_op_off;    /* [n_instrs+1] */
    const uint8_t *instr_n_defs;     /* [n_instrs] */
    const uint32_t *op_vreg;         /* [n_operands], each < n_vregs (n_vregs <= 65535) */
    const uint8_t *vreg_width;       /* [n_vregs], 1..255 */
} vl_program_desc;

/* One record per candidate (16 bytes). */
typedef struct {
    uint32_t flags;                /* VL_PASS or an OR of the violation bits */
    int32_t first_violation_instr; /* lowest instruction index carrying any violation; -1 if none */
    uint32_t conflict_pairs;       /* (instruction, definition, other vreg) range overlaps, summed */
    uint32_t bank_conflicts;       /* extra read cycles: per instruction, per bank, distinct source
                                      base registers beyond the first (bank model of Section 2) */
} vl_verdict;

typedef struct vl_program vl_program; /* opaque; owns device copies of the program and of its liveness */

/*
 * Validates the descriptor on the host and uploads it to `device`.
 * Errors: INVALID_ARG, MALFORMED_PROGRAM, UNSUPPORTED, CUDA.  *out is set only on VL_OK.
 */
int vl_program_create(const vl_program_desc *desc, int device, vl_program **out);

/* Frees every device and host resource of the handle.  NULL is accepted. */
void vl_program_destroy(vl_program *prog);

/* Sets a tunable; must precede vl_liveness.  Errors: INVALID_ARG. */
int vl_program_set_option(vl_program *prog, int option, uint32_t value);

/*
 * Liveness (what "overlapping life cycles" in Section 2 and "Safety" in Section 3.4
 * rest on): per-block read/write bitsets, backward dataflow to the least fixed point,
 * then the set of vregs live after every instruction as CSR lists (ascending ids),
 * plus the tables vl_verify consumes.  Stream order: the run is enqueued on an internal stream
 * of the device, behind everything `cuda_stream` (a cudaStream_t, may be NULL) holds at the call;
 * `cuda_stream` itself is NOT made to wait for it.  Every call of this library that reads the
 * results waits for the run where it needs them: vl_verify* on the device (its table kernel, which
 * reads the candidates and the program's operand tables only, runs beside the liveness kernels;
 * the kernels after it wait), vl_liveness_result, vl_verify_host, vl_diagnose and
 * vl_occupied_masks on the host.  A caller whose own kernels read the result arrays calls
 * vl_liveness_result after every run (it returns when the run has finished).
 * The first run of a handle (and the first after the chunk size changed) waits for the device
 * before returning, because list lengths and the status word are read back; it is the run that
 * reports NOT_STRICT or NO_CONVERGE, and the one that makes the operand tables (they depend on
 * the program alone and are kept).  Later runs recompute the liveness results on the device but
 * allocate from the remembered lengths and return without waiting: their outcome is checked by
 * the next call that uses the results, which may then return the error.  From the third such run
 * on the sequence of kernels is replayed as a CUDA graph (a recording of the library's own: do not
 * call vl_liveness while `cuda_stream` is itself being captured).
 * Errors: NOT_STRICT, NO_CONVERGE, UNSUPPORTED, CUDA.
 */
int vl_liveness(vl_program *prog, void *cuda_stream);

/*
 * vl_liveness for n independent programs (all on the device of the first) in one call: the
 * runs are spread over internal streams that fork from and join back into `cuda_stream` (unlike
 * a single vl_liveness, `cuda_stream` waits for them), so that the short kernels of different
 * programs run side by side.  `progs` is HOST memory.
 * Stops at the first error and returns it.  Errors: as vl_liveness, INVALID_ARG.
 */
int vl_liveness_batch(uint32_t n, vl_program *const *progs, void *cuda_stream);

/*
 * Device pointers to the liveness results; owned by the handle, valid until
 * vl_program_destroy or the next vl_liveness.  Any out pointer may be NULL.  Waits on the host
 * until the last liveness run of the handle has finished and returns its outcome.
 *   blk_live_in / blk_live_out : [n_blocks][ceil(n_vregs/32)] little-endian bitsets
 *   lo_off [n_instrs+1], lo [lo_len] : vregs live after each instruction, ascending
 */
int vl_liveness_result(const vl_program *prog, const uint32_t **blk_live_in, const uint32_t **blk_live_out,
                       const uint32_t **lo_off, const uint32_t **lo, uint64_t *lo_len);

/*
 * Checks K candidates.  d_cand is DEVICE memory, uint16, candidate-major:
 * d_cand[k * pitch_elems + o] is the physical register candidate k gives operand o.
 * Requirements: base 16-byte aligned, pitch_elems >= n_operands rounded up to 8,
 * pitch_elems % 8 == 0.  d_out is DEVICE memory for K records (4-byte aligned).
 * Buffers are borrowed for the call; the work is ordered after what `cuda_stream` holds at
 * the call, and what is enqueued on `cuda_stream` later is ordered after the work.  K == 0 is a no-op.
 * A call with more than one pass (VL_OPT_SUB_BATCH; the passes of a call are made equally long)
 * spreads its passes over internal streams of the device (VL_OPT_LANES) that fork from and join
 * back into `cuda_stream`, so that kernels of different passes run side by side; with
 * VL_OPT_LANES = 1 every kernel is enqueued on `cuda_stream` itself.
 * Host work of a call: the handle is modified (it owns the working memory of its calls).  The first
 * call on a handle, and a later one that needs larger working sets (more rows per pass, another
 * chunk size, more internal streams in use), allocates them with cudaMalloc and clears them, which
 * waits for the device: make one call of the intended size before timing or capturing.  A call that
 * fits the working sets allocates nothing and does not wait for the device, with one exception: the
 * first vl_verify* after a vl_liveness that returned early (see there) waits for that run's status
 * word, after its own kernels have been enqueued.  Each pass encodes one tensor-map descriptor for
 * the tiled copies on the host (no device work).
 *
 * Per candidate (Section 3.4): T[v] = register at the first occurrence of v;
 * Consistency: every occurrence equals T[v]; Realizability: at every definition
 * [T[v], T[v]+width) lies inside [0, P); Safety: at every definition of v the range of
 * v is disjoint from the range of every other vreg live after that instruction or
 * defined by it.  Bank tally per Section 2 with B banks.
 * UNSUPPORTED: P + widest vreg > 32768; the occupancy masks of one warp of the walk,
 * (P + widest vreg + 31) / 32 words for each of 64 candidates, do not fit the shared memory of an SM
 * (P up to about 28,000 fits); or the table of one candidate, 2 (n_vregs + 1) bytes, does not.
 * Errors: INVALID_ARG, LIVENESS_NOT_RUN, UNSUPPORTED, CUDA.
 */
int vl_verify(vl_program *prog, const uint16_t *d_cand, uint64_t K, uint64_t pitch_elems,
              vl_verdict *d_out, void *cuda_stream);

/*
 * Candidates in the form the paper's model emits them (Section 3.1: the allocation is generated per
 * basic block, as a dictionary from the block's virtual registers to physical registers; Section 3.2:
 * registers are renumbered per basic block, so one virtual register appears in the dictionaries of
 * every block that uses it).  A dictionary row holds one uint16 per (block, vreg occurring in the
 * block): blocks in program order, the vregs of a block in the order of their first occurrence in it
 * (definitions of an instruction before its reads; the paper fixes no order, this is the library's).
 * vl_dict_layout gives the layout: *n_entries columns, dict_off[n_blocks + 1] (first column of every
 * block) and dict_vreg[n_entries]; the arrays are HOST memory owned by the handle, valid until
 * vl_program_destroy.  Any out pointer may be NULL.
 */
int vl_dict_layout(const vl_program *prog, uint32_t *n_entries, const uint32_t **dict_off, const uint32_t **dict_vreg);

/*
 * vl_verify for K dictionary rows: d_dict[k * pitch_elems + e] is the register row k gives to
 * column e of the layout above (DEVICE memory, base 16-byte aligned, pitch_elems % 8 == 0 and at
 * least n_entries rounded up to 8).  Meaning: every occurrence of v inside block b carries the
 * register of column (b, v), and the row is checked as that per-occurrence assignment.  The table
 * value T[v] is the entry of the lowest block that uses v; Consistency (Section 3.4) compares the
 * entries of one vreg across blocks, and a differing entry is reported at the first instruction of
 * its block that touches the vreg; Realizability, Safety and the bank tally follow from T as in
 * vl_verify.  Same stream ordering, host work, limits and errors as vl_verify.
 */
int vl_verify_dict(vl_program *prog, const uint16_t *d_dict, uint64_t K, uint64_t pitch_elems, vl_verdict *d_out,
                   void *cuda_stream);

/*
 * The same check for n independent programs in one call (all on the device of the
 * first program): program j checks K[j] rows of d_cand[j] into d_out[j].  The arrays of
 * pointers and sizes are HOST memory.  Stream-ordered, no synchronisation.
 */
int vl_verify_batch(uint32_t n, vl_program *const *progs, const uint16_t *const *d_cand,
                    const uint64_t *K, const uint64_t *pitch_elems, vl_verdict *const *d_out,
                    void *cuda_stream);

/*
 * End-to-end form with HOST buffers: h_cand (K rows, same layout rules, ideally
 * pinned) is copied to the device in slabs through two staging buffers owned by the
 * handle, each slab is checked, and the verdicts are copied back (through pinned memory of the
 * handle) to h_out.  Copies and
 * kernels of successive slabs overlap on two internal streams; the call returns after
 * everything has finished (it synchronises).  `cuda_stream` orders the start of the work.
 * Errors: as vl_verify.
 */
int vl_verify_host(vl_program *prog, const uint16_t *h_cand, uint64_t K, uint64_t pitch_elems,
                   vl_verdict *h_out, void *cuda_stream);

/*
 * Optional hardware rules for the Realizability check (Section 1: register file sizes and reserved
 * registers; Section 3.2: scalar and vector register classes; Section 4.5: hardware rules on register
 * tuples).  With rules set, a definition of v violates Realizability (VL_OUT_OF_RANGE, reported at the
 * instruction of the definition) also when T[v] is not a multiple of vreg_align[v], when
 * [T[v], T[v]+width) is not inside [class_lo[c], class_hi[c]) for c = vreg_class[v], or when it holds a
 * reserved register.  Classes are ranges of the one register numbering 0..P-1; Safety and the bank
 * tally are unchanged (a misplaced tuple is compared with the others where it sits).
 * All pointers are HOST memory, read during the call; a NULL member switches that rule off.
 */
#define VL_MAX_CLASSES 8
typedef struct {
    const uint8_t *vreg_align;     /* [n_vregs], each >= 1 */
    const uint8_t *vreg_class;     /* [n_vregs], each < n_classes */
    uint32_t n_classes;            /* 1..VL_MAX_CLASSES when vreg_class is given */
    const uint32_t *class_lo;      /* [n_classes] */
    const uint32_t *class_hi;      /* [n_classes], class_lo <= class_hi <= P */
    const uint32_t *reserved_mask; /* ceil(P/32) words, bit (r & 31) of word r / 32: register r is reserved */
} vl_constraints;

/*
 * Sets (or, with rules == NULL or all members NULL, clears) the rules of the handle for later
 * vl_verify* calls.  Waits for the device, then replaces the handle's copies.
 * Errors: INVALID_ARG (alignment 0, class out of range, bad class range), CUDA.
 */
int vl_program_set_constraints(vl_program *prog, const vl_constraints *rules);

/*
 * Statistics of the re-sampling loop (Section 3.4, last paragraph: the model is sampled again until
 * a candidate passes or the attempts run out; Section 4: Pass@k, AvgTry, MaxTry).  The rows of a
 * verdict array are the attempts of one test case, in order.
 */
typedef struct {
    uint64_t first_pass; /* row of the first verdict with VL_PASS; K if there is none */
    uint64_t n_pass;     /* verdicts with VL_PASS among the K rows */
} vl_sample_stats;

#define VL_MAX_PASS_AT 8
typedef struct {
    uint64_t n_cases;                 /* test cases summarised */
    uint64_t n_solved;                /* test cases with a passing row */
    uint64_t sum_tries;               /* attempts up to and including the first passing one, summed over
                                         the solved test cases: AvgTry = sum_tries / n_solved */
    uint64_t max_tries;               /* the largest such number of attempts (MaxTry); 0 if none solved */
    uint64_t pass_at[VL_MAX_PASS_AT]; /* pass_at[j]: test cases solved within their first k[j] attempts
                                         (Pass@k[j] = pass_at[j] / n_cases); 0 for j >= n_k */
} vl_resample_summary;

/*
 * For each of n test cases: the record of d_out[j] (K[j] verdicts in DEVICE memory, 16-byte aligned,
 * as vl_verify wrote them) into d_stats[j]; then, unless d_summary is NULL, the summary of the n
 * records for the n_k <= VL_MAX_PASS_AT attempt limits k[].  d_out, K and k are HOST arrays, read
 * during the call; d_stats ([n]) and d_summary are DEVICE memory, 8-byte aligned, owned by the
 * caller.  A test case with K[j] == 0 counts as unsolved.  Stream-ordered on `cuda_stream` of
 * `device`, no synchronisation, no allocation.  Errors: INVALID_ARG, CUDA.
 */
int vl_resample_stats(int device, uint32_t n, const vl_verdict *const *d_out, const uint64_t *K, uint32_t n_k,
                      const uint32_t *k, vl_sample_stats *d_stats, vl_resample_summary *d_summary,
                      void *cuda_stream);

/*
 * The re-sampling loop with early exit: checks the rows of d_cand (as vl_verify) in batches of
 * batch_rows, in order, and stops after the first batch that holds a passing row.  *rows_checked
 * (HOST) receives the number of rows checked, a multiple of batch_rows or K; *first_pass (HOST) the
 * row of the first passing candidate, K if none passed.  Verdicts of the rows checked are in d_out
 * (16-byte aligned); those of later rows are not written.  The call waits for the stream after every
 * batch (the caller needs the answer to stop sampling); the first call allocates one record in
 * device and in pinned host memory.  Errors: as vl_verify.
 */
int vl_verify_until_pass(vl_program *prog, const uint16_t *d_cand, uint64_t K, uint64_t pitch_elems,
                         uint64_t batch_rows, vl_verdict *d_out, uint64_t *rows_checked, uint64_t *first_pass,
                         void *cuda_stream);

/*
 * Diagnostics of one candidate, as feedback for the sampler (Section 4.5 sorts failures into dataflow
 * and hardware-constraint violations; Section 6 proposes the verifier's findings as a training signal).
 * For the row d_row (DEVICE, n_operands entries): every Safety violation as a record (instruction,
 * defined vreg, other vreg) into d_conflicts (DEVICE, room for `cap` records, in no particular order;
 * records beyond `cap` are counted, not stored) with the total in *d_n_conflicts (DEVICE, 8-byte aligned;
 * equals the verdict's conflict_pairs); unless NULL, d_kinds[i] (DEVICE, n_instrs bytes) receives the OR
 * of the violation bits raised at instruction i (the lowest i with a bit is first_violation_instr) and
 * d_bank_hist[b] (DEVICE, B counters) the extra read cycles charged to bank b (their sum is
 * bank_conflicts).  Rules set with vl_program_set_constraints apply.  Not a hot path: one warp per
 * instruction over the live-after lists.  Stream-ordered, no synchronisation; the first call allocates
 * 8 * n_vregs bytes in the handle.  Errors: INVALID_ARG, LIVENESS_NOT_RUN, CUDA.
 */
typedef struct {
    uint32_t instr, vreg, other;
} vl_conflict;
int vl_diagnose(vl_program *prog, const uint16_t *d_row, uint64_t cap, vl_conflict *d_conflicts,
                uint64_t *d_n_conflicts, uint8_t *d_kinds, uint64_t *d_bank_hist, void *cuda_stream);

/*
 * Registers the definitions of every instruction must keep off, for decoding that masks out occupied
 * registers (Section 4.5, last paragraph).  For the row d_row (DEVICE, n_operands entries; a vreg that
 * has no register yet carries any value >= P, e.g. 0xFFFF, and contributes nothing):
 * d_masks[i * W + r / 32] bit (r & 31), W = ceil(P / 32), is set iff register r < P lies in the range of
 * a vreg that is live after instruction i and is not defined by i, or is reserved
 * (vl_program_set_constraints).  A definition of instruction i is safe iff its range touches no set bit
 * and no other definition of i.  d_masks is DEVICE memory for n_instrs * W words.  Stream-ordered, no
 * synchronisation; the first call allocates 8 * n_vregs + 8 bytes in the handle.
 * Errors: INVALID_ARG, LIVENESS_NOT_RUN, CUDA.
 */
int vl_occupied_masks(vl_program *prog, const uint16_t *d_row, uint32_t *d_masks, void *cuda_stream);

/*
 * Block-level liveness without any allocation.  (The paper has no counterpart; this exists for
 * hosts that cannot allocate device memory when they call in: a process that handed all of HBM to
 * its own pools at start-up, a plugin under a memory budget it does not control, or a loop that
 * cannot afford the device-wide synchronisation an allocation brings.)
 *
 * Computes the same live-in / live-out block bitsets as vl_liveness + vl_liveness_result, from a
 * program whose CSR arrays are already in DEVICE memory (same meaning and layout as the fields of
 * vl_program_desc; the program is not validated on the host, but an operand that names no vreg of
 * the program, or a successor that names no block, is skipped on the device and the call returns
 * VL_ERR_MALFORMED_PROGRAM), into the caller's DEVICE buffers d_live_in and d_live_out, each
 * [n_blocks][max(1, ceil(n_vregs/32))] 32-bit words.  d_succ may be NULL only for a program without
 * edges.  Nothing is checked for strictness here.
 *
 * The per-block read and write sets are kept in one fixed array inside the library,
 * VL_STATIC_SCRATCH_WORDS words (1 MiB) on every GPU that loads it, for the life of the process.
 * A program needs 2 * n_blocks * max(1, ceil(n_vregs/32)) of those words; a larger one is refused
 * with VL_ERR_UNSUPPORTED.  All calls on a device share the array and it keeps what the last call
 * left (each call rewrites every word it reads), so two calls whose kernels may overlap on the GPU
 * (different streams, different threads) race: serialise them.
 *
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress); make that
 * first call outside any stream capture.  The call launches on `cuda_stream`, then waits for it,
 * because the convergence status is read back.  It calls no cudaMalloc, cudaFree or other
 * allocating routine.
 * Errors: INVALID_ARG, UNSUPPORTED, MALFORMED_PROGRAM, NO_CONVERGE, CUDA.
 */
#define VL_STATIC_SCRATCH_WORDS (1u << 18)
int vl_block_liveness_static(int device, uint32_t n_blocks, uint32_t n_vregs, const uint32_t *d_block_instr_off,
                             const uint32_t *d_succ_off, const uint32_t *d_succ, const uint32_t *d_instr_op_off,
                             const uint8_t *d_instr_n_defs, const uint32_t *d_op_vreg, uint32_t *d_live_in,
                             uint32_t *d_live_out, void *cuda_stream);

/* Reads and clears the device-side status word of the handle's verify calls
 * (VL_OK or VL_ERR_DEVICE_WAIT).  Synchronises `cuda_stream`. */
int vl_verify_status(vl_program *prog, void *cuda_stream);

/* Number of kernels this library has launched in this process (all handles). */
uint64_t vl_kernel_launches(void);

/*
 * Device time of the verify kernels since the last call (or since VL_OPT_KERNEL_TIMING was set), summed over
 * the passes recorded (at most 4096): ms[0] table kernel (first occurrences, Consistency, Realizability, bank
 * tally), ms[1] occupancy walk (Safety), ms[2] verdict kernel, ms[3] exact recount.  ms is HOST memory for
 * 4 floats; *passes (HOST, may be NULL) receives the number of passes summed.  Kernels of different passes
 * may run side by side (VL_OPT_LANES), so the four sums can add up to more than the duration of the calls.
 * Waits for the last recorded event, then forgets the events.  Without the option everything is 0.  Errors: INVALID_ARG, CUDA.
 */
int vl_kernel_times(vl_program *prog, float ms[4], uint32_t *passes);

/* Last CUDA error code seen by the handle (0 if none). */
int vl_last_cuda_error(const vl_program *prog);

const char *vl_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* VERILOCC_H */
