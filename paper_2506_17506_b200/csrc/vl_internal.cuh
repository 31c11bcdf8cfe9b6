// Internal declarations shared by the translation units of libverilocc.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <vector>

#include "verilocc.h"

// ---- per-operand flag byte written by the liveness walk (device array opflags[n_operands])
enum : uint8_t {
    OPF_DEF = 1,    // operand is a definition
    OPF_KILL = 2,   // read: the value dies here (first read of the vreg in the instruction)
    OPF_DUP = 4,    // read: same vreg read earlier by this instruction
    OPF_ELIDE = 8,  // definition of a vreg the instruction also reads and that stays live:
                    //   occupancy unchanged, no walk event
    OPF_SET = 16,   // definition: becomes occupied (live after, or several defs in the instruction)
    OPF_POST = 32,  // definition: dead, released again after the instruction's definitions
    OPF_DEAD = 64   // definition: vreg not live after the instruction
};

enum : uint32_t { VINFO_OCCURS = 1u << 8, VINFO_DEFINED = 1u << 9 };

// ---- device status word bits (prog->d_status[0] liveness, d_status[1] verify)
enum : uint32_t {
    ST_NO_CONVERGE = 1u,
    ST_NOT_STRICT = 2u,
    ST_MANY_USES = 4u,      // some instruction reads more than 4 operands (bank tally takes the general path)
    ST_SIZE_OVERFLOW = 8u,  // a list length does not fit 32 bits
    ST_DEVICE_WAIT = 16u    // a bounded wait in a verify kernel ran out
};

#define VL_MAX_GROUP 8
#define VL_LANES 8  // internal streams that the passes of device-resident verify calls can be spread over
#define VL_LIVE_STREAM (VL_LANES + 2)  // index of the internal stream a single vl_liveness call runs on
#define VL_STREAMS (VL_LANES + 3)      // the lanes, two side streams of a liveness run, the liveness stream

// Device memory pool of a program handle: slabs are kept across calls, so that a repeated
// vl_liveness on the same handle allocates nothing.
struct VlArena {
    struct Slab { char *ptr; size_t size; };
    std::vector<Slab> slabs;
    size_t cur = 0, off = 0;
    cudaError_t alloc(void **out, size_t bytes)
    {
        bytes = (bytes + 64 + 255) & ~(size_t)255;
        for (; cur < slabs.size(); ++cur, off = 0)
            if (off + bytes <= slabs[cur].size) {
                *out = slabs[cur].ptr + off;
                off += bytes;
                return cudaSuccess;
            }
        Slab s{nullptr, bytes > ((size_t)4 << 20) ? bytes : ((size_t)4 << 20)};
        cudaError_t e = cudaMalloc((void **)&s.ptr, s.size);
        if (e != cudaSuccess) return e;
        slabs.push_back(s);
        cur = slabs.size() - 1;
        *out = s.ptr;
        off = bytes;
        return cudaSuccess;
    }
    void reset() { cur = 0; off = 0; }
    void release()
    {
        for (auto &s : slabs) cudaFree(s.ptr);
        slabs.clear();
        reset();
    }
};

struct vl_program {
    int device = 0;
    uint32_t nB = 0, nI = 0, V = 0, nO = 0, nE = 0, P = 0, B = 0;
    uint32_t Wv = 0;    // 32-bit words per vreg bitset
    uint32_t nOp8 = 0;  // n_operands rounded up to 8 (at least 8)
    uint32_t nOpT = 0;  // n_operands rounded up to 4096 (whole tiles of the eight-candidate table kernel), plus 4096
    uint32_t wmax = 1;  // widest vreg
    uint32_t chunk_instrs = 160;
    uint32_t group_opt = 0;

    // chunks: every chunk lies inside one block; pieces: every piece lies inside one chunk
    uint32_t nC = 0, nP = 0;
    uint32_t layout_chunk_instrs = 0;  // chunk size the device copies of the layout were made for (0: none)
    std::vector<uint32_t> h_blk_off, h_op_off;
    // list lengths of the last liveness run with this layout: the next run allocates from them
    bool sizes_known = false;
    uint64_t known_lo_len = 0, known_steps = 0, known_thn = 0, known_ls_len = 0;

    // device copies of the program
    uint32_t *d_blk_off = nullptr, *d_succ_off = nullptr, *d_succ = nullptr, *d_op_off = nullptr, *d_op_vreg = nullptr;
    uint8_t *d_ndefs = nullptr, *d_width = nullptr;
    uint32_t *d_chunk_i0 = nullptr, *d_chunk_i1 = nullptr, *d_chunk_blk = nullptr, *d_blk_chunk_off = nullptr;
    uint32_t *d_piece_i0 = nullptr, *d_piece_i1 = nullptr, *d_piece_chunk = nullptr, *d_chunk_piece_off = nullptr;

    // liveness results
    uint32_t *d_blk_in = nullptr, *d_blk_out = nullptr, *d_lo_off = nullptr, *d_lo = nullptr;
    uint64_t lo_len = 0;

    // tables consumed by the verify kernels
    uint16_t *d_vreg16 = nullptr;           // [nOp8 + 8] vreg id per operand (padding operands: id V)
    uint64_t *d_slotmeta = nullptr;         // [nOp8 / 8] per 8 operands: first-occurrence bits, bank compare masks
    // the same tables for rows in dictionary form (one column per (block, vreg of the block)); made once,
    // when the handle is created
    uint32_t nD = 0, nD8 = 0, nDT = 0;  // entries; rounded up to 8 (at least 8); to whole tiles plus one
    std::vector<uint32_t> h_dict_off, h_dict_vreg;
    uint16_t *d_dict_vreg16 = nullptr;
    uint64_t *d_dict_slotmeta = nullptr;
    uint4 *d_dict_opoff = nullptr;
    uint8_t *d_dict_first4 = nullptr;
    uint32_t *d_dict_instr = nullptr;     // [nD8] first instruction of the entry's block that touches its vreg
    uint4 *d_opoff = nullptr;               // [nOpT / 4] per 4 operands: byte offsets of their vregs' 16-byte table entries
    uint8_t *d_first4 = nullptr;            // [nOpT / 4] per 4 operands: first-occurrence bits
    uint8_t *d_opflags = nullptr;           // [nO]
    uint8_t *d_iflags = nullptr;            // [nI] 1 if the instruction has a definition the walk skips
    uint32_t *d_first_def_instr = nullptr;  // [V] lowest instruction defining v, 0xFFFFFFFF if none
    uint32_t *d_vinfo = nullptr;            // [V] width | VINFO_OCCURS | VINFO_DEFINED
    // optional hardware rules of the Realizability check (vl_program_set_constraints)
    uint4 *d_vcons = nullptr;               // [V] (class first | class end << 16, alignment, ceil(2^32 / alignment), 0); null = no rules
    uint16_t *d_rs_prefix = nullptr;        // [P+1] reserved registers below r; null = none reserved
    uint32_t *d_th_off = nullptr, *d_th = nullptr;  // per block: vregs occupied through the whole block
    // live-after lists without the block's through-set, for the recount: the list of instruction i of
    // block b is ls[lo_off[i] - ls_adj[b] - i * th_cnt[b] ...), |live-after| - th_cnt[b] entries
    uint32_t *d_ls = nullptr, *d_ls_adj = nullptr, *d_th_cnt = nullptr, *d_blk_th = nullptr;
    uint4 *d_el = nullptr;          // definitions without a walk event: {instruction, chunk, vreg, block}, any order
    uint32_t *d_el_count = nullptr;
    uint32_t th_len = 0;
    uint32_t *d_cev_off = nullptr;  // [nC+1] first walk event of each chunk (every chunk padded to 8 events)
    uint4 *d_ev = nullptr;          // walk events, 112 bytes per group of 8, chunk after chunk
    uint32_t ev_total = 0;
    // walk work items: a run of chunks of one block
    uint32_t nItems = 0;
    uint32_t *d_item_blk = nullptr, *d_item_c0 = nullptr, *d_item_c1 = nullptr;
    int bank_fast = 0;  // B in {1,2,4} and every instruction reads <= 4 distinct vregs
    int bank_many = 0;  // some instruction reads more than 4 distinct vregs
    uint2 *d_bank_list = nullptr;   // instructions with 2, 3, 4 distinct sources: their vreg ids, 16 bits each
    uint32_t bank_seg[4] = {0, 0, 0, 0};
    uint32_t threads_opt = 0;
    uint32_t prefetch_tiles = 3;
    uint32_t stagger_us = 12;     // start offset between the classes of the first wave of the table kernel (0 = none)
    int sm_count = 0;             // multiprocessors of the device (asked once)  // tiles the eight-candidate table kernel asks into L2 ahead of its copy ring
    uint32_t test_wait = 0;  // test hook of the table kernel's bounded wait (VL_OPT_TEST_WAIT)
    int use_th = 0;

    VlArena live_arena, tmp_arena;  // liveness results and tables / liveness working sets
    VlArena layout_arena;           // chunks, pieces, walk items
    uint32_t *d_status = nullptr;  // [16] device status words
    int last_cuda_error = 0;
    bool live_ok = false;
    // A repeated liveness run (same layout, lengths remembered) does not wait for the GPU: its status
    // word and list lengths are copied to pinned host memory behind the kernels, and the next call
    // that needs the results on the host side (vl_live_settle) waits for the copy and checks them.
    uint32_t *h_live = nullptr;      // pinned: [0] status, [2..9] four 64-bit totals
    cudaEvent_t ev_live = nullptr;
    bool live_pending = false;
    // vl_liveness runs on an internal stream behind what the caller's stream held when it was called;
    // the caller's stream is not made to wait.  Calls that read the results make their stream wait
    // for ev_live (vl_live_join); the table kernel, which reads the program's operand tables only,
    // runs beside the liveness kernels.
    bool live_deferred = false;
    cudaEvent_t ev_pre = nullptr;
    // The operand tables of the verify kernels (vreg per operand, first-occurrence bits, table
    // offsets, vreg descriptors, first definitions) depend on the program alone: they are made by the
    // first liveness run and kept (layout arena).
    bool tables_built = false;
    // the recorded form of a liveness run with settled layout and lengths (see vl_liveness_impl)
    cudaGraphExec_t live_graph = nullptr;
    uint64_t live_graph_launches = 0;
    uint32_t settled_runs = 0;
    int graph_opt = 1;

    // per-call working memory of vl_verify (one set per internal stream slot), grown on demand
    struct VScratch {
        uint16_t *tg = nullptr;      // [groups][V+1][64] tables, 64 candidates side by side
        uint32_t *cstate = nullptr;  // [rows][8]
        uint32_t *anom = nullptr;    // [rows][AW] chunks whose walk collided
        uint32_t *work = nullptr;    // [1 + rows] count, then candidates that need the exact recount
        uint32_t *racc = nullptr;    // [rows][4] recount accumulators: pairs, lowest instruction, bank tally, slices done
        uint32_t *grp_done = nullptr;  // walk thread blocks that have finished, per group of 64 candidates; then the groups' mark flags
        uint32_t *thm = nullptr;       // [groups][n_blocks][mask words][2][32] through-set masks
        uint64_t rows = 0, aw = 0, vregs = 0, chunks = 0;
    } vs[VL_LANES + 2];              // one per lane, then one per staging buffer of vl_verify_host
    uint32_t sub_batch = 5120;       // candidates per pass of the verify kernels
    uint32_t lanes_opt = 3;          // lanes in use (1 = everything in order on the caller's stream)
    cudaEvent_t ev_fork = nullptr, ev_join[VL_LANES] = {};
    cudaEvent_t ev_side[3] = {};     // fork and two joins of the side streams of a liveness run

    // opt-in per-kernel timing of vl_verify: five events per pass (before each of the four kernels, after the last)
    int ktime = 0;
    std::vector<cudaEvent_t> kt_ev;
    size_t kt_used = 0;

    // staging for vl_verify_host
    uint16_t *d_stage[2] = {nullptr, nullptr};
    vl_verdict *d_stage_out[2] = {nullptr, nullptr};
    uint64_t stage_rows = 0, stage_pitch = 0;
    vl_verdict *h_out_pinned = nullptr;  // verdicts of a vl_verify_host call on their way back
    uint64_t h_out_cap = 0;
    cudaStream_t h_streams[2] = {nullptr, nullptr};
    cudaEvent_t h_events[2] = {nullptr, nullptr};
    // one record for vl_verify_until_pass: device copy and its pinned landing place
    vl_sample_stats *d_rs = nullptr, *h_rs = nullptr;
    unsigned long long *d_diag_T = nullptr;  // [V] scratch of vl_diagnose: (first occurrence << 16) | value
    unsigned long long *d_diag_n = nullptr;  // one counter: scratch of vl_occupied_masks
};

extern std::atomic<uint64_t> g_vl_launches;

#define VL_CUDA(prog, call)                     \
    do {                                        \
        cudaError_t e__ = (call);               \
        if (e__ != cudaSuccess) {               \
            (prog)->last_cuda_error = (int)e__; \
            return VL_ERR_CUDA;                 \
        }                                       \
    } while (0)

int vl_liveness_impl(vl_program *p, cudaStream_t st);
int vl_verify_impl(vl_program *p, const uint16_t *d_cand, uint64_t K, uint64_t pitch, vl_verdict *d_out,
                   cudaStream_t st, int slot, bool dict = false);
int vl_verify_lanes(uint32_t nprog, vl_program *const *progs, const uint16_t *const *d_cand, const uint64_t *K,
                    const uint64_t *pitch, vl_verdict *const *d_out, cudaStream_t st, bool dict = false);
// The lane streams of the handle's device (created once per device; two side streams for liveness
// follow the VL_LANES lanes in the array) and the handle's fork / join events.
int vl_lane_streams(vl_program *p, cudaStream_t **lanes);
void vl_free_liveness(vl_program *p);
// Waits for a liveness run that is still in flight and checks its outcome; VL_OK if none is pending.
int vl_live_settle(vl_program *p);
int vl_live_join(vl_program *p, cudaStream_t st);  // st waits for the liveness run in flight, if any
// Multiprocessors of a device / of the handle's device (asked once).
int vl_device_sm_count(int device);
int vl_sm_count(vl_program *p);
void vl_drop_live_graph(vl_program *p);
