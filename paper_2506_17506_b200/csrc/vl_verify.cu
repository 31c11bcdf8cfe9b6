// The verify path: four kernels per pass over at most `sub_batch` candidates.
//
// k_tables8  one thread block per 8 candidates, packed side by side (16 bytes per vreg).  A producer warp
//            streams the 8 rows with tiled bulk copies into a shared-memory ring (completion on
//            mbarriers); 16 consumer warps build the vreg -> register table T in shared memory from first
//            occurrences and compare every other occurrence with T (Consistency).  Then the block sweeps
//            the vregs ([T, T+width) inside the register file: Realizability; T to global memory, 64
//            candidates side by side per vreg) and tallies bank conflicts over the instructions with
//            2..4 distinct sources.  k_tables<G,NT> (G = 4, 2, 1 candidates per block, block barrier per
//            tile) serves programs whose 16-byte tables do not fit an SM.
// k_through  the occupancy masks of every block's through-set (vregs occupied through the whole block),
//            per candidate, in the walk's layout.
// k_walk     two candidates per lane, one warp per chunk of instructions: the program's precompiled
//            event stream is the same for all lanes, the occupancy bitmasks of a lane sit in shared
//            memory at [word][slot][lane] (Safety).  A chunk whose walk sees no collision provably
//            has no overlap.  The thread block that ends a group of 64 candidates writes the verdicts
//            of its clean candidates and lists the others for the recount.
// k_recount  candidates with a collision are recounted exactly from the per-instruction live-after
//            lists: work items (a piece of a colliding chunk, a block whose through-set collided, the
//            bank tally of a candidate) taken from a shared cursor, long items first.
#include <cuda.h>

#include <algorithm>
#include <cstring>
#include <mutex>

#include "vl_internal.cuh"

#define MAX_STAGES 4
#define TGW 64  // candidates side by side per vreg in the tables handed from the table kernel to the walk
#define WALK_WARPS 8
#define RC_THREADS 256

// per-candidate state between the kernels (8 words)
enum { CS_FLAGS = 0, CS_FIRST = 1, CS_BANK = 2, CS_NOUT = 3, CS_OUTV = 4, CS_OUTRAW = 5, CS_WALK = 6, CS_THCOL = 7 };
enum : uint32_t { WALK_ANOM = 1u, WALK_FULL = 2u };

struct TParams {
    uint32_t nI, V, nO, nOp8, P, Bmask, ntiles;
    int bank_fast;
    const uint16_t *vreg16;
    const uint64_t *slotmeta;
    const uint32_t *vinfo, *first_def_instr, *op_off;
    const uint2 *bank_list;
    uint32_t bank_seg[4];  // entries with n = 2, 3, 4 distinct sources: [seg[n-2], seg[n-1])
    uint32_t bank_total;   // distinct sources summed over the listed instructions
    const uint16_t *cand;
    uint64_t K, pitch;
    uint16_t *tg;
    uint32_t *cstate;
    uint32_t *status;
    uint32_t NS, off_region, off_misc;
    // per-pass state this kernel clears for the kernels after it
    uint32_t AW;
    uint32_t *anom, *racc, *grp_done, *work;
    // optional hardware rules: per vreg (first | end << 16 of its class's registers, alignment,
    // ceil(2^32 / alignment)), and
    // the number of reserved registers below every register
    const uint4 *vcons;
    const uint16_t *rs_prefix;
    // the eight-candidate kernel: per 4 operands the byte offsets of their vregs' table entries and
    // their first-occurrence bits
    const uint4 *opoff;
    const uint8_t *first4;
    // dictionary rows: the instruction a Consistency violation of entry e is reported at (null: the rows
    // hold one column per operand, and the instruction is the one the operand belongs to)
    const uint32_t *entry_instr;
    uint32_t tg_rows;     // k_tables8: vregs per bulk store of the table (rows of the box of the tg tensor)
    uint32_t *grp_flag;   // per group of 64 candidates: some table entry carries the straddle mark
    uint32_t test_wait;   // test hook: the wait for tile 0 polls a barrier nothing completes, with a short limit
    uint32_t pf;          // tiles asked into L2 ahead of the copy ring
    uint32_t stagger_ns, stagger_blocks;  // k_tables8: start offset between the four classes of the first wave's blocks
    // the rows as a 3-D tensor [candidate][chunk of 256 operands][256]: nfull whole chunks per row; the
    // operands from tail_start on (fewer than 256) come by plain bulk copies into a buffer of their own
    uint32_t nfull, tail_start, tail_tile, off_tail;
};

struct TMisc {
    unsigned long long bar[MAX_STAGES];
    unsigned long long bar_never;  // initialised, never completed: what the test hook waits on
    unsigned long long bar_tail;   // the operands behind the last whole chunk of 256
    unsigned long long empty[MAX_STAGES];  // k_tables8: every consumer warp has read the stage
    unsigned long long stored[2];          // k_tables8: every consumer warp has stored its first occurrences of a tile (by tile parity)
    uint32_t flags[VL_MAX_GROUP], minop[VL_MAX_GROUP], minR[VL_MAX_GROUP], bank[VL_MAX_GROUP];
    uint32_t nout[VL_MAX_GROUP], out_v[VL_MAX_GROUP], out_raw[VL_MAX_GROUP];
    uint32_t abort_flag;
    uint32_t marks;  // bit g: a table entry of candidate g carries the straddle mark
};

struct WParams {
    uint32_t V, P, nB, nC, Wp, AW, use_th, wmax;
    uint64_t K;
    const uint32_t *th_off, *th, *cev_off;
    uint32_t *thm;  // [groups][nB][Wp][2][32] through-set masks (k_through -> k_walk)
    const uint4 *ev;
    const uint16_t *tg;
    uint32_t ev_cap;  // events a warp stages at a time (multiple of 8)
    uint32_t *cstate, *anom;
    uint32_t *grp_flag;  // per group: set by the table kernel when a walked candidate has a marked entry
    // hand-over to k_recount by the last thread block of each group of 64 candidates
    int list_all;
    const uint32_t *chunk_blk;
    uint32_t *grp_done, *work, *racc;
    vl_verdict *out;
};

struct RParams {
    uint32_t nI, V, B, nB, nC, AW;
    int bank_fast;
    uint64_t K;
    const uint32_t *vinfo, *chunk_i0, *chunk_i1, *chunk_blk, *blk_chunk_off, *th_off, *th, *op_off, *op_vreg, *lo_off, *lo;
    const uint8_t *ndefs, *width, *opflags, *iflags;
    const uint16_t *tg;
    const uint32_t *cstate, *anom;
    uint32_t *racc;
    const uint2 *bank_list;
    uint32_t bank_seg[4];
    uint32_t *work;
    vl_verdict *out;
    uint32_t *status;
    const uint4 *el;           // the definitions the walk skips: {instruction, chunk, vreg, block}
    const uint32_t *el_count;
    const uint32_t *ls, *ls_adj, *th_cnt;  // live-after lists without the through-sets (see vl_program)
    uint32_t R;                            // registers covered by the recount's through-set counters
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(unsigned long long *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok;
}
// Bulk async copy global -> this block's shared memory, completion counted on `bar`.
// dst, src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, unsigned long long *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// Tiled copy of one box of a 3-D tensor (coordinates innermost first) into this block's shared memory,
// completion counted on `bar` with the full size of the box (elements outside the tensor arrive as
// zeros).  dst 128-byte aligned; the innermost coordinate times the element size a multiple of 16.
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *tm, uint32_t x, uint32_t y, uint32_t z,
                                            unsigned long long *bar, unsigned long long policy)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;" ::"r"(
            smem_u32(dst)),
        "l"(tm), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
// L2 policy for data that is read once: first in line for eviction, so that it does not push out what
// other kernels are about to read again.
// Tiled bulk store of one box from shared memory (elements outside the tensor are not written); completion is
// tracked by the issuing thread's bulk async-groups.
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *tm, uint32_t x, uint32_t y, uint32_t z, const void *src)
{
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
                 ::"l"(tm), "r"(x), "r"(y), "r"(z), "r"(smem_u32(src))
                 : "memory");
}

__device__ __forceinline__ unsigned long long l2_policy_evict_first()
{
    unsigned long long policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}
// Asks for one box of the tensor to be brought into L2.
__device__ __forceinline__ void tma_prefetch_3d(const CUtensorMap *tm, uint32_t x, uint32_t y, uint32_t z)
{
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(tm), "r"(x), "r"(y), "r"(z)
                 : "memory");
}

// ------------------------------------------------------------- packed table access
// In shared memory T holds, per vreg, the G candidates' registers side by side (16 bits each).
template <int G>
__device__ __forceinline__ uint64_t t_load(const uint16_t *Tt, uint32_t v)
{
    if constexpr (G == 4) {
        uint2 x = *reinterpret_cast<const uint2 *>(Tt + (size_t)v * 4);
        return (uint64_t)x.x | ((uint64_t)x.y << 32);
    } else if constexpr (G == 2) {
        return *reinterpret_cast<const uint32_t *>(Tt + (size_t)v * 2);
    } else {
        return Tt[v];
    }
}
template <int G>
__device__ __forceinline__ void t_store(uint16_t *Tt, uint32_t v, uint64_t x)
{
    if constexpr (G == 4) {
        *reinterpret_cast<uint2 *>(Tt + (size_t)v * 4) = make_uint2((uint32_t)x, (uint32_t)(x >> 32));
    } else if constexpr (G == 2) {
        *reinterpret_cast<uint32_t *>(Tt + (size_t)v * 2) = (uint32_t)x;
    } else {
        Tt[v] = (uint16_t)x;
    }
}
__device__ __forceinline__ uint32_t pk_get(uint64_t x, int g) { return (uint32_t)(x >> (16 * g)) & 0xFFFFu; }

__device__ __forceinline__ bool ranges_overlap(uint32_t a, uint32_t wa, uint32_t b, uint32_t wb)
{
    return a < b + wb && b < a + wa;
}

// Hardware rules on where the tuples may sit (alignment, registers of the vreg's class, reserved
// registers) for the G candidates of a block: a sweep of its own over the vregs, run only for
// programs that have rules, four vregs per thread and round so that the loads of a round are in
// flight together.  Kept out of line, so the kernel's other phases keep their registers.  The
// remainder uses the reciprocal the host stored (exact for 16-bit values and alignments up to 255).
template <int G, int NT>
__device__ __noinline__ void rules_sweep(const uint4 *vcons, const uint16_t *rs_prefix, const uint32_t *vinfo,
                                         const uint32_t *first_def_instr, uint32_t V, uint32_t P,
                                         const uint16_t *Tt, TMisc *M)
{
    for (uint32_t v0 = threadIdx.x; v0 < V; v0 += 4 * NT) {
        uint4 vc[4];
        uint32_t vi[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t v = v0 + u * NT;
            vc[u] = v < V ? vcons[v] : make_uint4(0, 0, 0, 0);
            vi[u] = v < V ? vinfo[v] : 0u;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t v = v0 + u * NT;
            if (v >= V || !(vi[u] & VINFO_DEFINED)) continue;
            const uint32_t clo = vc[u].x & 0xFFFFu, chi = vc[u].x >> 16, al = vc[u].y, recip = vc[u].z;
            const uint32_t w = vi[u] & 0xFFu;
            const uint64_t tt = t_load<G>(Tt, v);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const uint32_t tv = pk_get(tt, g);
                bool bad = (al > 1 && tv != __umulhi(tv, recip) * al) || tv < clo || tv + w > chi;
                if (!bad && rs_prefix) bad = rs_prefix[min(tv + w, P)] != rs_prefix[min(tv, P)];
                if (bad) {
                    atomicOr(&M->flags[g], (uint32_t)VL_OUT_OF_RANGE);
                    atomicMin(&M->minR[g], first_def_instr[v]);
                }
            }
        }
    }
}

// =========================================================================== k_tables
template <int G, int NT>
__global__ void __launch_bounds__(NT) k_tables(const TParams q)
{
    constexpr uint32_t TILE = NT * 8;  // operands per tile and candidate
    constexpr uint32_t STAGE_BYTES = TILE * 2;
    extern __shared__ __align__(16) unsigned char smem[];
    uint16_t *Tt = reinterpret_cast<uint16_t *>(smem);
    unsigned char *region = smem + q.off_region;
    uint16_t *Hb = reinterpret_cast<uint16_t *>(region);  // [V] after the rows have been streamed: bank nibbles
    TMisc *M = reinterpret_cast<TMisc *>(smem + q.off_misc);

    const uint32_t tid = threadIdx.x, lane = tid & 31;
    const uint64_t k0 = (uint64_t)blockIdx.x * G;
    const uint16_t *rows[G];
#pragma unroll
    for (int g = 0; g < G; ++g) rows[g] = q.cand + min(k0 + g, q.K - 1) * q.pitch;

    if (tid < G) {
        M->flags[tid] = 0; M->minop[tid] = 0xFFFFFFFFu; M->minR[tid] = 0xFFFFFFFFu; M->bank[tid] = 0;
        M->nout[tid] = 0; M->out_v[tid] = 0; M->out_raw[tid] = 0;
    }
    if (tid == 0) {
        M->abort_flag = 0;
        for (uint32_t s = 0; s < q.NS; ++s) mbar_init(&M->bar[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // state of this pass that the walk and the recount update with atomics starts at zero
    for (uint32_t j = tid; j < G * q.AW; j += NT) q.anom[k0 * q.AW + j] = 0;
    if (tid < G * 4) q.racc[k0 * 4 + tid] = 0;
    if (tid == 0 && (k0 & (TGW - 1)) == 0) q.grp_done[k0 / TGW] = 0;
    if (tid == 0 && blockIdx.x == 0) { q.work[0] = 0; q.work[1] = 0; q.work[2] = 0; }  // item count and the recount's two cursors
    __syncthreads();

    // The ring stage and the barrier phase of the current tile are kept as running counters (stage
    // wraps at NS, the phase flips with it): no division in the loop.
    auto issue_tile = [&](uint32_t t, uint32_t stage) {
        const uint32_t bytes = min(TILE, q.nOp8 - t * TILE) * 2;
        mbar_expect_tx(&M->bar[stage], bytes * G);
#pragma unroll
        for (int g = 0; g < G; ++g)
            bulk_g2s(region + (size_t)(stage * G + g) * STAGE_BYTES, rows[g] + (size_t)t * TILE, bytes, &M->bar[stage]);
    };
    if (tid == 0)
        for (uint32_t t = 0; t < q.NS && t < q.ntiles; ++t) issue_tile(t, t);

    // Per tile: load it from the ring and store its first occurrences to the table, barrier, compare
    // every occurrence with the table.  The compare of tile t may overlap the stores of tile t+1 by
    // faster threads: those are first occurrences of other vregs.
    auto wait_tile = [&](uint32_t stage, uint32_t parity) {  // bounded wait
        uint32_t spins = 0;
        const uint32_t limit = *(volatile uint32_t *)&M->abort_flag ? 64u : (1u << 22);
        while (!mbar_try_wait(&M->bar[stage], parity)) {
            if (++spins > limit) {
                M->abort_flag = 1;
                atomicOr(q.status, ST_DEVICE_WAIT);
                break;
            }
        }
    };
    // loads this thread's 8 operands x G candidates of tile t and transposes them to
    // "G candidates side by side per operand"; stores the first occurrences
    auto load_tile = [&](uint32_t t, uint32_t stage, uint64_t (&pc)[8], uint32_t (&vj)[8], const uint4 &v4,
                         uint32_t first) {
        const bool act = t * TILE + tid * 8 < q.nOp8;
        uint32_t r[G][4];
        if (act) {
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const uint4 c4 =
                    *reinterpret_cast<const uint4 *>(region + (size_t)(stage * G + g) * STAGE_BYTES + tid * 16);
                r[g][0] = c4.x; r[g][1] = c4.y; r[g][2] = c4.z; r[g][3] = c4.w;
            }
        } else {
#pragma unroll
            for (int g = 0; g < G; ++g) r[g][0] = r[g][1] = r[g][2] = r[g][3] = 0;
        }
        const uint32_t vr[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int k = j >> 1;
            const uint32_t sel = (j & 1) ? 0x7632u : 0x5410u;
            if constexpr (G == 4) {
                pc[j] = (uint64_t)__byte_perm(r[0][k], r[1][k], sel) |
                        ((uint64_t)__byte_perm(r[2][k], r[3][k], sel) << 32);
            } else if constexpr (G == 2) {
                pc[j] = __byte_perm(r[0][k], r[1][k], sel);
            } else {
                pc[j] = (j & 1) ? (r[0][k] >> 16) : (r[0][k] & 0xFFFFu);
            }
            vj[j] = (j & 1) ? (vr[k] >> 16) : (vr[k] & 0xFFFFu);
        }
        if (act) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if ((first >> j) & 1) t_store<G>(Tt, vj[j], pc[j]);
        }
    };
    // every occurrence of tile t against the table (a first occurrence trivially matches; padding
    // operands beyond n_operands are left out)
    auto compare_tile = [&](uint32_t t, const uint64_t (&pc)[8], const uint32_t (&vj)[8]) {
        const uint32_t o_base = t * TILE + tid * 8;
        if (o_base >= q.nOp8) return;
        uint64_t acc = 0;
        if (o_base + 8 <= q.nO) {
#pragma unroll
            for (int j = 0; j < 8; ++j) acc |= t_load<G>(Tt, vj[j]) ^ pc[j];
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (o_base + j < q.nO) acc |= t_load<G>(Tt, vj[j]) ^ pc[j];
        }
        if (acc) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (o_base + j >= q.nO) continue;
                const uint64_t d = t_load<G>(Tt, vj[j]) ^ pc[j];
#pragma unroll
                for (int g = 0; g < G; ++g)
                    if (pk_get(d, g)) {
                        atomicOr(&M->flags[g], (uint32_t)VL_INCONSISTENT);
                        atomicMin(&M->minop[g], o_base + j);
                    }
            }
        }
    };
    // operand metadata (vreg ids, first-occurrence bits) comes from global memory, fetched one tile ahead
    auto load_meta = [&](uint32_t t, uint4 &v4, uint32_t &first) {
        const uint32_t o = t * TILE + tid * 8;
        if (t < q.ntiles && o < q.nOp8) {
            v4 = *reinterpret_cast<const uint4 *>(q.vreg16 + o);
            first = (uint32_t)q.slotmeta[o >> 3] & 0xFFu;
        } else {
            v4 = make_uint4(0, 0, 0, 0);
            first = 0;
        }
    };
    {
        uint64_t pc[8];
        uint32_t vj[8];
        uint4 m_v4, m2_v4;
        uint32_t m_first, m2_first;
        load_meta(0, m_v4, m_first);
        uint32_t stage = 0, parity = 0;
        for (uint32_t t = 0; t < q.ntiles; ++t) {
            load_meta(t + 1, m2_v4, m2_first);
            wait_tile(stage, parity);
            load_tile(t, stage, pc, vj, m_v4, m_first);
            __syncthreads();
            if (tid == 0 && t + q.NS < q.ntiles) issue_tile(t + q.NS, stage);  // the stage just read is free again
            compare_tile(t, pc, vj);
            m_v4 = m2_v4;
            m_first = m2_first;
            if (++stage == q.NS) { stage = 0; parity ^= 1; }
        }
    }
    __syncthreads();

    // ---- one sweep over the vregs: the table goes to global memory (64 candidates side by side per
    // vreg; the spare entry V, looked up by no-op events, as 0) and [T, T+width) is checked against the
    // register file (Realizability)
    {
        const uint64_t grp = k0 / TGW;
        const uint32_t l0 = (uint32_t)(k0 & (TGW - 1));
        uint16_t *dst = q.tg + grp * (uint64_t)(q.V + 1) * TGW + l0;
        uint32_t vis_next[8];  // the vreg descriptors of the next round are fetched during the current one
#pragma unroll
        for (int u = 0; u < 8; ++u) vis_next[u] = tid + u * NT < q.V ? q.vinfo[tid + u * NT] : 0u;
        for (uint32_t v0 = tid; v0 <= q.V; v0 += 8 * NT) {
            uint32_t vis[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                vis[u] = vis_next[u];
                const uint32_t vn = v0 + 8 * NT + u * NT;
                vis_next[u] = vn < q.V ? q.vinfo[vn] : 0u;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const uint32_t v = v0 + u * NT, vi = vis[u];
                if (v > q.V) break;
                const uint64_t tt = v < q.V ? t_load<G>(Tt, v) : 0ull;
                uint32_t lo = (uint32_t)tt, hi = (uint32_t)(tt >> 32);
                if (q.bank_fast && v < q.V) {  // one-hot bank nibbles of the G candidates
                    uint32_t h = (1u << (lo & q.Bmask));
                    if constexpr (G >= 2) h |= 16u << ((lo >> 16) & q.Bmask);
                    if constexpr (G == 4) h |= (256u << (hi & q.Bmask)) | (4096u << ((hi >> 16) & q.Bmask));
                    Hb[v] = (uint16_t)h;
                }
                {   // bit 15 of an entry handed to the walk marks a range that reaches into the next 32-bit
                    // word of the occupancy mask (every in-file register number is below 2^15):
                    // per 16-bit entry bit 15 := ((register & 31) + width > 32); 0x7FDF = 0x8000 - 33
                    const uint32_t wc = (vi & 0xFFu) * 0x10001u + 0x7FDF7FDFu;
                    lo = (lo & 0x7FFF7FFFu) | (((lo & 0x001F001Fu) + wc) & 0x80008000u);
                    hi = (hi & 0x7FFF7FFFu) | (((hi & 0x001F001Fu) + wc) & 0x80008000u);
                }
                if constexpr (G == 4) {
                    *reinterpret_cast<uint2 *>(dst + (size_t)v * TGW) = make_uint2(lo, hi);
                } else if constexpr (G == 2) {
                    *reinterpret_cast<uint32_t *>(dst + (size_t)v * TGW) = lo;
                } else {
                    dst[(size_t)v * TGW] = (uint16_t)lo;
                }
                if (!(vi & VINFO_OCCURS)) continue;
                const uint32_t w = vi & 0xFFu;
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const uint32_t tv = pk_get(tt, g);
                    if (tv + w > q.P) {
                        if (vi & VINFO_DEFINED) {
                            atomicOr(&M->flags[g], (uint32_t)VL_OUT_OF_RANGE);
                            atomicMin(&M->minR[g], q.first_def_instr[v]);
                        }
                        if (atomicAdd(&M->nout[g], 1u) == 0) { M->out_v[g] = v; M->out_raw[g] = tv; }
                    }
                }
            }
        }
    }
    if (q.vcons) rules_sweep<G, NT>(q.vcons, q.rs_prefix, q.vinfo, q.first_def_instr, q.V, q.P, Tt, M);

    __syncthreads();
    // ------------------------------- bank tally: instructions with 2..4 distinct sources.
    // Distinct vregs read by one instruction are live together, so a candidate whose walk sees no
    // collision has them on distinct registers, and its tally for one instruction is the number of
    // sources minus the number of banks they touch.  Hb[v] holds, per candidate, the bank of T[v]
    // as a one-hot nibble: the banks touched are the bits of the OR over the sources (list entries
    // repeat their first source in unused slots).  The bits are counted with carry-save adders, 8
    // entries per round.  Candidates with a collision get the general tally in k_recount.
    if (q.bank_fast) {
        auto csa = [](uint32_t &h, uint32_t &l, uint32_t a, uint32_t b, uint32_t c) {
            const uint32_t u = a ^ b;
            h = (a & b) | (u & c);
            l = u ^ c;
        };
        // per nibble of the low 16 bits: its population count, as four byte fields (nibbles 0, 2, 1, 3)
        auto nibble_counts = [](uint32_t x) -> uint32_t {
            uint32_t y = (x & 0x0F0Fu) | ((x & 0xF0F0u) << 12);
            y = y - ((y >> 1) & 0x55555555u);
            return (y & 0x33333333u) + ((y >> 2) & 0x33333333u);
        };
        auto field = [](uint32_t c, int g) -> uint32_t { return (c >> ((g & 1) * 16 + (g >> 1) * 8)) & 0xFFu; };
        uint32_t ones = 0, twos = 0, fours = 0, acc8 = 0, rounds = 0;
        uint32_t sum[G];
#pragma unroll
        for (int g = 0; g < G; ++g) sum[g] = 0;
        const uint32_t n_ent = q.bank_seg[3];
        uint2 ids_next[8];  // list entries of the next round are fetched during the current one
#pragma unroll
        for (int u = 0; u < 8; ++u) ids_next[u] = tid + u * NT < n_ent ? q.bank_list[tid + u * NT] : make_uint2(0, 0);
        for (uint32_t e0 = tid; e0 < n_ent; e0 += 8 * NT) {
            uint2 ids[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                ids[u] = ids_next[u];
                const uint32_t en = e0 + 8 * NT + u * NT;
                ids_next[u] = en < n_ent ? q.bank_list[en] : make_uint2(0, 0);
            }
            uint32_t x[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const uint32_t o = (uint32_t)Hb[ids[u].x & 0xFFFFu] | Hb[ids[u].x >> 16] | Hb[ids[u].y & 0xFFFFu] |
                                   Hb[ids[u].y >> 16];
                x[u] = e0 + u * NT < n_ent ? o : 0u;
            }
            uint32_t ta, tb, fa, fb, eights;
            csa(ta, ones, ones, x[0], x[1]);
            csa(tb, ones, ones, x[2], x[3]);
            csa(fa, twos, twos, ta, tb);
            csa(ta, ones, ones, x[4], x[5]);
            csa(tb, ones, ones, x[6], x[7]);
            csa(fb, twos, twos, ta, tb);
            csa(eights, fours, fours, fa, fb);
            acc8 += nibble_counts(eights);
            if (++rounds == 32) {  // the byte fields of acc8 hold at most 4 per round
#pragma unroll
                for (int g = 0; g < G; ++g) sum[g] += 8u * field(acc8, g);
                acc8 = 0;
                rounds = 0;
            }
        }
        const uint32_t c4 = nibble_counts(fours), c2 = nibble_counts(twos), c1 = nibble_counts(ones);
#pragma unroll
        for (int g = 0; g < G; ++g) {
            uint32_t x = sum[g] + 8u * field(acc8, g) + 4u * field(c4, g) + 2u * field(c2, g) + field(c1, g);
#pragma unroll
            for (int d = 16; d; d >>= 1) x += __shfl_xor_sync(0xffffffffu, x, d);
            if (lane == 0 && x) atomicAdd(&M->bank[g], x);
        }
    }
    __syncthreads();

    // ------------------------------------------------- hand-over to the walk
    // One vreg sticking out of the file cannot overlap another one out there: the walk sees it
    // parked at P (bits beyond P are padding).  Two or more: the candidate is recounted in full.
    // (such a candidate does not take part in the walk: it gets its table back without the marks)
#pragma unroll
    for (int g = 0; g < G; ++g) {
        if (M->nout[g] < 2) continue;
        uint16_t *col = q.tg + (k0 / TGW) * (uint64_t)(q.V + 1) * TGW + (uint32_t)(k0 & (TGW - 1)) + g;
        for (uint32_t v = tid; v < q.V; v += NT) col[(size_t)v * TGW] = (uint16_t)pk_get(t_load<G>(Tt, v), g);
    }
    if (tid < G && M->nout[tid] == 1 && M->out_raw[tid] >= q.P) {
        const uint32_t ov = M->out_v[tid];
        const uint32_t mark = ((q.P & 31u) + (q.vinfo[ov] & 0xFFu) > 32u) ? 0x8000u : 0u;
        q.tg[(k0 / TGW) * (uint64_t)(q.V + 1) * TGW + (size_t)ov * TGW + (uint32_t)(k0 & (TGW - 1)) + tid] = (uint16_t)(q.P | mark);
    }
    if (tid < G && k0 + tid < q.K) {
        const uint32_t g = tid;
        uint32_t first = 0xFFFFFFFFu;
        if (M->minop[g] != 0xFFFFFFFFu && q.entry_instr) {
            // dictionary rows: entries are in block order and, inside a block, in order of first
            // occurrence, so the lowest violating entry is also the lowest violating instruction
            first = q.entry_instr[M->minop[g]];
        } else if (M->minop[g] != 0xFFFFFFFFu) {  // operand -> instruction: last i with op_off[i] <= operand
            const uint32_t o = M->minop[g];
            uint32_t lo_i = 0, hi_i = q.nI;  // invariant: op_off[lo_i] <= o < op_off[hi_i]
            while (hi_i - lo_i > 1) {
                const uint32_t mid = (lo_i + hi_i) >> 1;
                if (q.op_off[mid] <= o) lo_i = mid; else hi_i = mid;
            }
            first = lo_i;
        }
        uint32_t *cs = q.cstate + (k0 + g) * 8;
        cs[CS_FLAGS] = M->flags[g];
        cs[CS_FIRST] = min(first, M->minR[g]);
        cs[CS_BANK] = q.bank_fast ? q.bank_total - M->bank[g] : 0u;
        cs[CS_NOUT] = M->nout[g];
        cs[CS_OUTV] = M->out_v[g];
        cs[CS_OUTRAW] = M->out_raw[g];
        cs[CS_WALK] = M->nout[g] >= 2 ? WALK_FULL : 0u;
        cs[CS_THCOL] = 0;
    }
    // this kernel does not keep track of marked entries: its groups take the walk's checking path
    if (tid == 0) atomicOr(&q.grp_flag[k0 / TGW], 1u);
}

// =========================================================================== k_tables8
// The table kernel with eight candidates per thread block: a table entry is 16 bytes (the eight
// candidates' registers of one vreg), so that one shared-memory load serves eight operand checks.
// A thread takes 4 operands x 8 candidates per tile (one 8-byte load per row from the copy ring),
// transposes them with byte permutes, stores first occurrences, and compares the occurrences of the
// tile before (whose first occurrences a barrier has already ordered) while the current tile's loads
// are in flight: one barrier per tile, no dependent wait behind it.
__device__ __forceinline__ uint32_t pk8_get(const uint4 &x, int g)
{
    const uint32_t w = (g >> 1) == 0 ? x.x : ((g >> 1) == 1 ? x.y : ((g >> 1) == 2 ? x.z : x.w));
    return (g & 1) ? (w >> 16) : (w & 0xFFFFu);
}

template <int NT>
__device__ __noinline__ void rules_sweep8(const uint4 *vcons, const uint16_t *rs_prefix, const uint32_t *vinfo,
                                          const uint32_t *first_def_instr, uint32_t V, uint32_t P, const uint4 *T,
                                          TMisc *M)
{
    for (uint32_t v = threadIdx.x; v < V; v += NT) {
        const uint32_t vi = vinfo[v];
        if (!(vi & VINFO_DEFINED)) continue;
        const uint4 vc = vcons[v];
        const uint32_t clo = vc.x & 0xFFFFu, chi = vc.x >> 16, al = vc.y, recip = vc.z, w = vi & 0xFFu;
        const uint4 tt = T[v];
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            const uint32_t tv = pk8_get(tt, g);
            bool bad = (al > 1 && tv != __umulhi(tv, recip) * al) || tv < clo || tv + w > chi;
            if (!bad && rs_prefix) bad = rs_prefix[min(tv + w, P)] != rs_prefix[min(tv, P)];
            if (bad) {
                atomicOr(&M->flags[g], (uint32_t)VL_OUT_OF_RANGE);
                atomicMin(&M->minR[g], first_def_instr[v]);
            }
        }
    }
}

template <int NT>
__global__ void __launch_bounds__(NT + 32, 1) k_tables8(const TParams q, const __grid_constant__ CUtensorMap tm,
                                                          const __grid_constant__ CUtensorMap tmg)
{
    constexpr int G = 8;
    constexpr uint32_t TILE = NT * 4;  // operands per tile and candidate
    constexpr uint32_t ROW_BYTES = TILE * 2, STAGE_BYTES = ROW_BYTES * G;
    constexpr uint32_t CH = TILE / 256;      // chunks of 256 operands per tile
    constexpr uint32_t TAIL_ROW_BYTES = 512;
    extern __shared__ __align__(16) unsigned char smem[];
    uint4 *T = reinterpret_cast<uint4 *>(smem);  // [V + 1]
    unsigned char *region = smem + q.off_region;
    uint32_t *Hb = reinterpret_cast<uint32_t *>(region);  // [V] after the rows have been streamed: bank nibbles
    unsigned char *tailbuf = smem + q.off_tail;           // [G][TAIL_ROW_BYTES]
    TMisc *M = reinterpret_cast<TMisc *>(smem + q.off_misc);

    const uint32_t tid = threadIdx.x, lane = tid & 31;
    const uint64_t k0 = (uint64_t)blockIdx.x * G;
    // The thread blocks of a wave would otherwise run in step: all of them stream (HBM saturated) and
    // then all of them sweep (HBM idle).  The first wave of a call starts in four classes a quarter of a
    // block's time apart; later blocks start when earlier ones end, so the offsets persist.
    if (q.stagger_ns && blockIdx.x < q.stagger_blocks && (blockIdx.x & 3u)) {
        if (tid == 0) {
            unsigned long long t0, t1;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
            const unsigned long long until = t0 + (unsigned long long)(blockIdx.x & 3u) * q.stagger_ns;
            do {
                __nanosleep(2000);
                asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
            } while (t1 < until && t1 - t0 < 1000000ull);  // (never longer than a millisecond)
        }
        __syncthreads();
    }
    const uint16_t *rows[G];
#pragma unroll
    for (int g = 0; g < G; ++g) rows[g] = q.cand + min(k0 + g, q.K - 1) * q.pitch;

    if (tid < G) {
        M->flags[tid] = 0; M->minop[tid] = 0xFFFFFFFFu; M->minR[tid] = 0xFFFFFFFFu; M->bank[tid] = 0;
        M->nout[tid] = 0; M->out_v[tid] = 0; M->out_raw[tid] = 0;
    }
    if (tid == 0) {
        M->abort_flag = 0;
        M->marks = 0;
        for (uint32_t s = 0; s < q.NS; ++s) { mbar_init(&M->bar[s], 1); mbar_init(&M->empty[s], NT / 32); }
        mbar_init(&M->stored[0], NT / 32);
        mbar_init(&M->stored[1], NT / 32);
        mbar_init(&M->bar_never, 1);
        mbar_init(&M->bar_tail, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        T[q.V] = make_uint4(0, 0, 0, 0);  // the spare entry: what padding operands are compared with
    }
    // state of this pass that the walk and the recount update with atomics starts at zero
    for (uint32_t j = tid; j < G * q.AW; j += NT) q.anom[k0 * q.AW + j] = 0;
    if (tid < G * 4) q.racc[k0 * 4 + tid] = 0;
    if (tid == 0 && (k0 & (TGW - 1)) == 0) q.grp_done[k0 / TGW] = 0;
    if (tid == 0 && blockIdx.x == 0) { q.work[0] = 0; q.work[1] = 0; q.work[2] = 0; }  // item count and the recount's two cursors
    __syncthreads();

    // A tile is one box of the row tensor: 8 candidates x CH chunks x 256 operands, one copy.  (Boxes
    // that reach past the last whole chunk, or past the last candidate, are filled up with zeros.)
    // Warp NT/32 is the producer: it refills a stage of the ring as soon as every consumer warp has
    // read it.  The consumer warps are not held together by a block barrier per tile; what orders
    // them is one counting barrier per tile parity, "the first occurrences of tile t are stored",
    // on which a warp arrives after its stores and waits one tile later, before it compares tile t.
    auto wait_bar = [&](unsigned long long *bar, uint32_t parity) {
        // Bounded wait.  When it runs out the block raises the status bit and carries on with short
        // waits (its results are garbage, every index still in bounds); the producer issues no
        // further copies and, before the block returns, waits again for the copies it did issue.
        if (mbar_try_wait(bar, parity)) return;
        uint32_t spins = 0;
        const uint32_t limit = *(volatile uint32_t *)&M->abort_flag ? 64u : (1u << 20);
        while (!mbar_try_wait(bar, parity)) {
            if (++spins > limit) {
                M->abort_flag = 1;
                atomicOr(q.status, ST_DEVICE_WAIT);
                break;
            }
        }
    };
    if (tid >= NT) {  // ------------------------------------------------------------ producer warp
        if (lane == 0) {
            const uint32_t tail_bytes = (q.nOp8 - q.tail_start) * 2;
            if (tail_bytes) {
                mbar_expect_tx(&M->bar_tail, tail_bytes * G);
#pragma unroll
                for (int g = 0; g < G; ++g)
                    bulk_g2s(tailbuf + g * TAIL_ROW_BYTES, rows[g] + q.tail_start, tail_bytes, &M->bar_tail);
            }
            uint32_t issued = 0;  // tiles issued so far, in order
            uint32_t stage = 0, parity = 0;
            // the rows are read once: they should not push the tables written for the walk out of L2
            const unsigned long long stream_once = l2_policy_evict_first();
            for (uint32_t t = 0; t < q.ntiles; ++t) {
                if (t >= q.NS) {  // the stage still holds tile t - NS: wait until the 16 warps have read it
                    wait_bar(&M->empty[stage], parity ^ 1u);
                    if (*(volatile uint32_t *)&M->abort_flag) break;
                }
                issued = t + 1;
                if (t * CH < q.nfull) {  // (a tile of nothing but tail operands has no box)
                    mbar_expect_tx(&M->bar[stage], STAGE_BYTES);
                    tma_load_3d(region + (size_t)stage * STAGE_BYTES, &tm, 0, t * CH, (uint32_t)k0, &M->bar[stage], stream_once);
                }
                if (++stage == q.NS) { stage = 0; parity ^= 1; }
            }
            if (*(volatile uint32_t *)&M->abort_flag) {
                // a wait ran out: give the copies that were issued their time before the block (and its
                // shared memory) goes away
                for (uint32_t s = 0; s < q.NS; ++s) {
                    if (issued <= s) continue;
                    uint32_t t_last = s + (issued - 1 - s) / q.NS * q.NS;  // the last tile issued into stage s
                    if (t_last * CH >= q.nfull) {
                        if (t_last < q.NS) continue;
                        t_last -= q.NS;
                    }
                    uint32_t spins = 0;
                    while (!mbar_try_wait(&M->bar[s], (t_last / q.NS) & 1u) && ++spins < (1u << 20)) {}
                }
                if (tail_bytes) {
                    uint32_t spins = 0;
                    while (!mbar_try_wait(&M->bar_tail, 0) && ++spins < (1u << 20)) {}
                }
            }
        }
    } else {  // ---------------------------------------------------------------------- consumer warps
        const uint32_t spare_off = q.V * 16u;
        const uint4 *opoff = q.opoff + tid;
        const uint8_t *first4 = q.first4 + tid;
        // every occurrence of a tile against the table (a first occurrence trivially matches; padding
        // operands were zeroed and name the all-zero spare entry)
        auto compare = [&](const uint4 (&pc)[4], const uint4 &off, uint32_t o_base) {
            const uint32_t of[4] = {off.x, off.y, off.z, off.w};
            uint4 x[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) x[j] = *reinterpret_cast<const uint4 *>(smem + of[j]);
            uint32_t acc = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                acc |= (x[j].x ^ pc[j].x) | (x[j].y ^ pc[j].y) | (x[j].z ^ pc[j].z) | (x[j].w ^ pc[j].w);
            if (acc) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t d[4] = {x[j].x ^ pc[j].x, x[j].y ^ pc[j].y, x[j].z ^ pc[j].z, x[j].w ^ pc[j].w};
#pragma unroll
                    for (int g = 0; g < G; ++g)
                        if ((g & 1) ? (d[g >> 1] >> 16) : (d[g >> 1] & 0xFFFFu)) {
                            atomicOr(&M->flags[g], (uint32_t)VL_INCONSISTENT);
                            atomicMin(&M->minop[g], o_base + j);
                        }
                }
            }
        };
        auto transpose = [&](const uint2 (&r)[G], uint4 (&pc)[4]) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t sel = (j & 1) ? 0x7632u : 0x5410u;
                uint32_t w[4];
#pragma unroll
                for (int m = 0; m < 4; ++m)
                    w[m] = (j < 2) ? __byte_perm(r[2 * m].x, r[2 * m + 1].x, sel) : __byte_perm(r[2 * m].y, r[2 * m + 1].y, sel);
                pc[j] = make_uint4(w[0], w[1], w[2], w[3]);
            }
        };
        auto store_first = [&](const uint4 (&pc)[4], const uint4 &off, uint32_t first) {
            const uint32_t of[4] = {off.x, off.y, off.z, off.w};
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if ((first >> j) & 1) *reinterpret_cast<uint4 *>(smem + of[j]) = pc[j];
        };
        // the warp has read its part of a stage / has stored its first occurrences of a tile
        auto warp_arrive = [&](unsigned long long *bar) {
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
        };
        uint32_t stage = 0, parity = 0;
        const uint32_t last = q.ntiles - 1;
        // thread i asks for line i % (ROW_BYTES / 128) of row i / (ROW_BYTES / 128) of a tile
        const unsigned char *pf_ptr = nullptr;
        if (q.pf && tid < G * (ROW_BYTES / 128))
            pf_ptr = reinterpret_cast<const unsigned char *>(q.cand + min(k0 + tid / (ROW_BYTES / 128), q.K - 1) * q.pitch) +
                     (tid % (ROW_BYTES / 128)) * 128;
        // operand metadata is fetched two tiles ahead (the arrays are padded to whole tiles, and one
        // tile more is readable behind them)
        uint4 off_n = opoff[0], off_n2 = opoff[NT];
        uint32_t first_n = first4[0], first_n2 = first4[NT];
        // one whole tile (not the last): load and transpose, store first occurrences, compare the tile before
        auto step = [&](uint32_t t, uint4 (&pc)[4], uint4 &off, const uint4 (&ppc)[4], const uint4 &poff) {
            off = off_n;
            const uint32_t first = first_n;
            off_n = off_n2;
            first_n = first_n2;
            off_n2 = opoff[(size_t)(t + 2) * NT];
            first_n2 = first4[(size_t)(t + 2) * NT];
            // The ring holds too few bytes to cover the latency of HBM by itself: the lines of a tile
            // further ahead are asked into L2 (one 128-byte line per thread), so that the ring's
            // copies come from there.
            if (pf_ptr && t + q.pf < last) asm volatile("prefetch.global.L2 [%0];" ::"l"(pf_ptr + (size_t)(t + q.pf) * ROW_BYTES));
            wait_bar(&M->bar[stage], parity);
            uint2 r[G];
            const unsigned char *src = region + (size_t)stage * STAGE_BYTES + tid * 8;
#pragma unroll
            for (int g = 0; g < G; ++g) r[g] = *reinterpret_cast<const uint2 *>(src + g * ROW_BYTES);
            transpose(r, pc);
            warp_arrive(&M->empty[stage]);
            store_first(pc, off, first);
            warp_arrive(&M->stored[t & 1]);
            if (t) wait_bar(&M->stored[(t - 1) & 1], ((t - 1) >> 1) & 1u);
            compare(ppc, poff, (t - 1) * TILE + tid * 4);
            if (++stage == q.NS) { stage = 0; parity ^= 1; }
        };
        uint4 pcA[4], pcB[4], offA, offB;
#pragma unroll
        for (int j = 0; j < 4; ++j) pcB[j] = make_uint4(0, 0, 0, 0);
        offB = make_uint4(spare_off, spare_off, spare_off, spare_off);  // "the tile before tile 0": zeros against the spare entry
        if (q.test_wait) {  // test hook: this wait runs out
            uint32_t spins = 0;
            while (!mbar_try_wait(&M->bar_never, 0)) {
                if (++spins > (1u << 16)) { M->abort_flag = 1; atomicOr(q.status, ST_DEVICE_WAIT); break; }
            }
        }
        uint32_t t = 0;
        for (; t + 2 <= last; t += 2) {
            step(t, pcA, offA, pcB, offB);
            step(t + 1, pcB, offB, pcA, offA);
        }
        if (t < last) {  // an odd number of whole tiles before the last: keep "the tile before" in B
            step(t, pcA, offA, pcB, offB);
#pragma unroll
            for (int j = 0; j < 4; ++j) pcB[j] = pcA[j];
            offB = offA;
            ++t;
        }
        {   // the last tile: it may hold the row's tail (from its own buffer) and operands beyond the row
            const uint32_t o_base = last * TILE + tid * 4;
            offA = off_n;
            const uint32_t first = first_n;
            uint2 r[G];
            if (o_base >= q.tail_start) {  // (a whole warp: the tail starts at a multiple of 256)
                if (o_base < q.nOp8) {     // the tail buffer ends where the rows end; beyond it there is padding only
                    wait_bar(&M->bar_tail, 0);
                    const unsigned char *src = tailbuf + (o_base - q.tail_start) * 2;
#pragma unroll
                    for (int g = 0; g < G; ++g) r[g] = *reinterpret_cast<const uint2 *>(src + g * TAIL_ROW_BYTES);
                } else {
#pragma unroll
                    for (int g = 0; g < G; ++g) r[g] = make_uint2(0, 0);
                }
            } else {
                wait_bar(&M->bar[stage], parity);
                const unsigned char *src = region + (size_t)stage * STAGE_BYTES + tid * 8;
#pragma unroll
                for (int g = 0; g < G; ++g) r[g] = *reinterpret_cast<const uint2 *>(src + g * ROW_BYTES);
            }
            transpose(r, pcA);
#pragma unroll
            for (int j = 0; j < 4; ++j)  // operands beyond n_operands compare as zero against the spare entry
                if (o_base + j >= q.nO) pcA[j] = make_uint4(0, 0, 0, 0);
            store_first(pcA, offA, first);
            warp_arrive(&M->stored[last & 1]);
            if (last) wait_bar(&M->stored[(last - 1) & 1], ((last - 1) >> 1) & 1u);
            compare(pcB, offB, (last - 1) * TILE + tid * 4);
            wait_bar(&M->stored[last & 1], (last >> 1) & 1u);
            compare(pcA, offA, o_base);
        }
    }
    __syncthreads();

    // ---- first sweep over the vregs: the one-hot bank nibbles of the 8 candidates go to Hb, and
    // [T, T+width) is checked against the register file (Realizability).
    // (From here on the producer warp only keeps the block's barriers company.)
    if (tid < NT) {
        uint32_t vis_next[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) vis_next[u] = tid + u * NT < q.V ? q.vinfo[tid + u * NT] : 0u;
        for (uint32_t v0 = tid; v0 < q.V; v0 += 4 * NT) {
            uint32_t vis[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                vis[u] = vis_next[u];
                const uint32_t vn = v0 + 4 * NT + u * NT;
                vis_next[u] = vn < q.V ? q.vinfo[vn] : 0u;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t v = v0 + u * NT, vi = vis[u];
                if (v >= q.V) break;
                const uint4 tt = T[v];
                const uint32_t x[4] = {tt.x, tt.y, tt.z, tt.w};
                if (q.bank_fast) {
                    uint32_t h = 0;
#pragma unroll
                    for (int m = 0; m < 4; ++m)
                        h |= ((1u << (x[m] & q.Bmask)) << (8 * m)) | ((16u << ((x[m] >> 16) & q.Bmask)) << (8 * m));
                    Hb[v] = h;
                }
                if (!(vi & VINFO_OCCURS)) continue;
                // quick test for "all eight inside the file": with c = 0x7FFF - (P - width) added to an
                // entry below 2^15, bit 15 of the sum is set iff entry + width > P; entries at or above
                // 2^15 are outside any file this kernel accepts.  The exact test runs only if a bit shows.
                const uint32_t w = vi & 0xFFu;
                uint32_t f = 1;
                if (w <= q.P) {
                    const uint32_t c2 = (0x7FFFu - (q.P - w)) * 0x10001u;
                    f = (((x[0] + c2) | x[0]) | ((x[1] + c2) | x[1]) | ((x[2] + c2) | x[2]) | ((x[3] + c2) | x[3])) & 0x80008000u;
                }
                if (f) {
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const uint32_t tv = pk8_get(tt, g);
                        if (tv + w > q.P) {
                            if (vi & VINFO_DEFINED) {
                                atomicOr(&M->flags[g], (uint32_t)VL_OUT_OF_RANGE);
                                atomicMin(&M->minR[g], q.first_def_instr[v]);
                            }
                            if (atomicAdd(&M->nout[g], 1u) == 0) { M->out_v[g] = v; M->out_raw[g] = tv; }
                        }
                    }
                }
            }
        }
    }
    if (q.vcons && tid < NT) rules_sweep8<NT>(q.vcons, q.rs_prefix, q.vinfo, q.first_def_instr, q.V, q.P, T, M);
    __syncthreads();

    // ---- second sweep, in place: entries whose range reaches into the next 32-bit word of an occupancy
    // mask get bit 15.  The entries of a candidate with two or more vregs outside the register file stay as
    // they are (it is not walked; the full recount reads them as plain numbers).
    if (tid < NT) {
        uint32_t keep[4];  // 16-bit fields of the candidates whose entries stay as they are
#pragma unroll
        for (int m = 0; m < 4; ++m)
            keep[m] = (M->nout[2 * m] >= 2 ? 0xFFFFu : 0u) | (M->nout[2 * m + 1] >= 2 ? 0xFFFF0000u : 0u);
        uint32_t mk = 0, mk2 = 0, mk3 = 0, mk4 = 0;
        uint32_t vis_next[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) vis_next[u] = tid + u * NT < q.V ? q.vinfo[tid + u * NT] : 0u;
        for (uint32_t v0 = tid; v0 < q.V; v0 += 4 * NT) {
            uint32_t vis[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                vis[u] = vis_next[u];
                const uint32_t vn = v0 + 4 * NT + u * NT;
                vis_next[u] = vn < q.V ? q.vinfo[vn] : 0u;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t v = v0 + u * NT, vi = vis[u];
                if (v >= q.V) break;
                if (!(vi & VINFO_OCCURS)) continue;  // (never looked up)
                const uint4 tt = T[v];
                const uint32_t x[4] = {tt.x, tt.y, tt.z, tt.w};
                // bit 15 := ((register & 31) + width > 32), per 16-bit entry; 0x7FDF = 0x8000 - 33
                const uint32_t wc = (vi & 0xFFu) * 0x10001u + 0x7FDF7FDFu;
                uint32_t o[4], diff = 0;
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    const uint32_t marked = (x[m] & 0x7FFF7FFFu) | (((x[m] & 0x001F001Fu) + wc) & 0x80008000u);
                    o[m] = (marked & ~keep[m]) | (x[m] & keep[m]);
                    diff |= o[m] ^ x[m];
                }
                if (diff) T[v] = make_uint4(o[0], o[1], o[2], o[3]);
                mk |= o[0] & ~keep[0]; mk2 |= o[1] & ~keep[1]; mk3 |= o[2] & ~keep[2]; mk4 |= o[3] & ~keep[3];
            }
        }
        const uint32_t mkw[4] = {mk, mk2, mk3, mk4};
        uint32_t bits = 0;
#pragma unroll
        for (int m = 0; m < 4; ++m) bits |= ((mkw[m] >> 15) & 1u) << (2 * m) | ((mkw[m] >> 31) & 1u) << (2 * m + 1);
        bits = __reduce_or_sync(0xffffffffu, bits);
        if (lane == 0 && bits) atomicOr(&M->marks, bits);
        // the consumers go on to the bank tally (it reads Hb only); the producer warp waits for all of them here
        asm volatile("bar.arrive 1, %0;" ::"r"(NT + 32) : "memory");
    }
    // The table goes to global memory, 64 candidates side by side per vreg (this block's 8 are 16 bytes of
    // every 128): tiled bulk stores of up to 256 vregs each, carried out by the copy engine while the block
    // tallies bank conflicts.  (Rows past the spare entry V are clipped by the tensor.)  Issuing a store holds
    // its thread for thousands of cycles: the lanes of the producer warp, idle since the last tile, issue them.
    bool stored = false;  // this thread has bulk stores under way
    if (tid >= NT) {
        asm volatile("bar.sync 1, %0;" ::"r"(NT + 32) : "memory");
        // a single out-of-file vreg is parked at register P (the walk's masks have spare bits there)
        if (lane < G && M->nout[lane] == 1 && M->out_raw[lane] >= q.P) {
            const uint32_t ov = M->out_v[lane];
            const uint32_t mark = ((q.P & 31u) + (q.vinfo[ov] & 0xFFu) > 32u) ? 0x8000u : 0u;
            reinterpret_cast<uint16_t *>(T + ov)[lane] = (uint16_t)(q.P | mark);
            if (mark) atomicOr(&M->marks, 1u << lane);
        }
        __syncwarp();
        if (lane * q.tg_rows <= q.V) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            const uint32_t x0 = (uint32_t)(k0 & (TGW - 1)), z0 = (uint32_t)(k0 / TGW);
            for (uint32_t v0 = lane * q.tg_rows; v0 <= q.V; v0 += 32 * q.tg_rows) tma_store_3d(&tmg, x0, v0, z0, T + v0);
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            stored = true;
        }
    }

    // ---- bank tally over the instructions with 2..4 distinct sources (see k_tables): the banks an
    // instruction touches are the bits of the OR of its sources' nibbles, counted with carry-save adders
    if (q.bank_fast && tid < NT) {
        auto csa = [](uint32_t &h, uint32_t &l, uint32_t a, uint32_t b, uint32_t c) {
            const uint32_t u = a ^ b;
            h = (a & b) | (u & c);
            l = u ^ c;
        };
        // population count of each of the 8 nibbles, as byte fields: even nibbles and odd nibbles
        auto nib_even = [](uint32_t y) -> uint32_t { return y & 0x0F0F0F0Fu; };
        auto nib_odd = [](uint32_t y) -> uint32_t { return (y >> 4) & 0x0F0F0F0Fu; };
        auto nib_counts = [](uint32_t x) -> uint32_t {
            const uint32_t y = x - ((x >> 1) & 0x55555555u);
            return (y & 0x33333333u) + ((y >> 2) & 0x33333333u);
        };
        uint32_t ones = 0, twos = 0, fours = 0, acc_e = 0, acc_o = 0, rounds = 0;
        uint32_t sum[G];
#pragma unroll
        for (int g = 0; g < G; ++g) sum[g] = 0;
        auto flush = [&](uint32_t weight) {
#pragma unroll
            for (int g = 0; g < G; ++g) sum[g] += weight * ((((g & 1) ? acc_o : acc_e) >> (8 * (g >> 1))) & 0xFFu);
            acc_e = 0; acc_o = 0;
        };
        const uint32_t n_ent = q.bank_seg[3];
        uint2 ids_next[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) ids_next[u] = tid + u * NT < n_ent ? q.bank_list[tid + u * NT] : make_uint2(0, 0);
        for (uint32_t e0 = tid; e0 < n_ent; e0 += 8 * NT) {
            uint2 ids[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                ids[u] = ids_next[u];
                const uint32_t en = e0 + 8 * NT + u * NT;
                ids_next[u] = en < n_ent ? q.bank_list[en] : make_uint2(0, 0);
            }
            uint32_t x[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const uint32_t o = Hb[ids[u].x & 0xFFFFu] | Hb[ids[u].x >> 16] | Hb[ids[u].y & 0xFFFFu] | Hb[ids[u].y >> 16];
                x[u] = e0 + u * NT < n_ent ? o : 0u;
            }
            uint32_t ta, tb, fa, fb, eights;
            csa(ta, ones, ones, x[0], x[1]);
            csa(tb, ones, ones, x[2], x[3]);
            csa(fa, twos, twos, ta, tb);
            csa(ta, ones, ones, x[4], x[5]);
            csa(tb, ones, ones, x[6], x[7]);
            csa(fb, twos, twos, ta, tb);
            csa(eights, fours, fours, fa, fb);
            const uint32_t c8 = nib_counts(eights);
            acc_e += nib_even(c8);
            acc_o += nib_odd(c8);
            if (++rounds == 32) {  // the byte fields hold at most 4 per round
                flush(8u);
                rounds = 0;
            }
        }
        flush(8u);
        uint32_t c = nib_counts(fours);
        acc_e = nib_even(c); acc_o = nib_odd(c);
        flush(4u);
        c = nib_counts(twos);
        acc_e = nib_even(c); acc_o = nib_odd(c);
        flush(2u);
        c = nib_counts(ones);
        acc_e = nib_even(c); acc_o = nib_odd(c);
        flush(1u);
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const uint32_t x = __reduce_add_sync(0xffffffffu, sum[g]);
            if (lane == 0 && x) atomicAdd(&M->bank[g], x);
        }
    }
    __syncthreads();

    // ------------------------------------------------- hand-over to the walk (see k_tables)
    if (tid < G && k0 + tid < q.K) {
        const uint32_t g = tid;
        uint32_t first = 0xFFFFFFFFu;
        if (M->minop[g] != 0xFFFFFFFFu && q.entry_instr) {
            // dictionary rows: entries are in block order and, inside a block, in order of first
            // occurrence, so the lowest violating entry is also the lowest violating instruction
            first = q.entry_instr[M->minop[g]];
        } else if (M->minop[g] != 0xFFFFFFFFu) {  // operand -> instruction: last i with op_off[i] <= operand
            const uint32_t o = M->minop[g];
            uint32_t lo_i = 0, hi_i = q.nI;  // invariant: op_off[lo_i] <= o < op_off[hi_i]
            while (hi_i - lo_i > 1) {
                const uint32_t mid = (lo_i + hi_i) >> 1;
                if (q.op_off[mid] <= o) lo_i = mid; else hi_i = mid;
            }
            first = lo_i;
        }
        uint32_t *cs = q.cstate + (k0 + g) * 8;
        cs[CS_FLAGS] = M->flags[g];
        cs[CS_FIRST] = min(first, M->minR[g]);
        cs[CS_BANK] = q.bank_fast ? q.bank_total - M->bank[g] : 0u;
        cs[CS_NOUT] = M->nout[g];
        cs[CS_OUTV] = M->out_v[g];
        cs[CS_OUTRAW] = M->out_raw[g];
        cs[CS_WALK] = M->nout[g] >= 2 ? WALK_FULL : 0u;
        cs[CS_THCOL] = 0;
        // a candidate that is walked and has a marked entry sends its group of 64 down the walk's
        // checking path
        if (M->nout[g] < 2 && ((M->marks >> g) & 1u)) atomicOr(&q.grp_flag[k0 / TGW], 1u);
    }
    // the bulk stores read the table from shared memory: the block stays until they are done
    if (stored) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v)
{
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t atom_xor_shared(uint32_t addr, uint32_t v)
{
    uint32_t old;
    asm volatile("atom.shared.xor.b32 %0, [%1], %2;" : "=r"(old) : "r"(addr), "r"(v) : "memory");
    return old;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ void finish_candidate(uint64_t k, uint32_t nC, uint32_t AW, int list_all, const uint32_t *cstate,
                                 const uint32_t *anom, const uint32_t *__restrict__ chunk_blk, uint32_t *work,
                                 uint32_t *racc, vl_verdict *out);

// An event group in shared memory is 112 bytes: off[8] (byte offset of the vreg's table row),
// toggle[8], test[8] (32-bit masks), wl[8] (16 bit).  Constant offsets go into the instruction.
template <int OFF>
__device__ __forceinline__ uint4 lds128_at(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4 + %5];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(addr), "n"(OFF)
                 : "memory");
    return v;
}

// A lane of the walk carries two candidates, 2 * lane and 2 * lane + 1 of its group of 64: their
// table entries sit side by side (one 32-bit load per event), their occupancy masks in shared memory
// at [word][slot 0 / 1][lane] (bank = lane for both).

// Table entries (this lane's two candidates) of the 8 vregs of the event group at shared address ga.
__device__ __forceinline__ void fetch_group(uint32_t ga, const unsigned char *tgb, uint32_t (&t)[8])
{
    const uint4 a = lds128_at<0>(ga), b = lds128_at<16>(ga);
    const uint32_t off[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        // base + offset as one multiply-add: the integer ALU pipe is the walk's bottleneck, the
        // multiply-add pipe has room.  The tables were written by the kernel before this one.
        unsigned long long addr;
        asm("mad.wide.u32 %0, %1, 1, %2;" : "=l"(addr) : "r"(off[u]), "l"(tgb));
        asm("ld.global.nc.u32 %0, [%1];" : "=r"(t[u]) : "l"(addr));
    }
}

// What a lane knows about one of its candidates: whether it is walked at all, and the address
// arithmetic that keeps a candidate that is not walked (its table may hold anything) inside the mask.
struct WalkSlot {
    uint32_t alive;  // 1 if walked, else 0: shifted to the range's position it gives the bit masks, or nothing
    uint32_t amask;  // slot 0: 0x7FE0 if walked else 0; slot 1: 2048 if walked else 0 (see apply_group)
};

// Applies the 8 events of the group at shared address ga to the occupancy masks of this lane's two
// candidates; viol collects the occupied bits that a test found.  Toggling returns the old word:
// occupied and released are both a toggle as long as no collision has been seen (after one, the
// chunk is recounted exactly anyway).  The caller vouches that no range of the group reaches into
// the next 32-bit word for any walked candidate and that none is wider than 32 registers: every
// event is one atomic per candidate.  Masks and addresses are computed with multiply-adds where
// possible, to spare the integer ALU pipe.
__device__ __forceinline__ void apply_group(uint32_t ga, const uint32_t (&t)[8], uint32_t occ_addr, const WalkSlot &A,
                                            const WalkSlot &B, uint32_t &violA, uint32_t &violB)
{
#pragma unroll
    for (int h = 0; h < 2; ++h) {  // the masks of four events at a time: fewer registers held
        const uint4 z4 = h ? lds128_at<48>(ga) : lds128_at<32>(ga), y4 = h ? lds128_at<80>(ga) : lds128_at<64>(ga);
        const uint32_t hz[4] = {z4.x, z4.y, z4.z, z4.w}, hy[4] = {y4.x, y4.y, y4.z, y4.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t t2 = t[4 * h + u];
            uint32_t a, mz, my;
            {   // slot 0: register = low half; its mask word (register / 32) is 256 bytes wide per word
                const uint32_t p2 = __funnelshift_l(0u, A.alive, t2);
                asm("mad.lo.u32 %0, %1, 8, %2;" : "=r"(a) : "r"(t2 & A.amask), "r"(occ_addr));
                asm("mul.lo.u32 %0, %1, %2;" : "=r"(mz) : "r"(hz[u]), "r"(p2));
                asm("mul.lo.u32 %0, %1, %2;" : "=r"(my) : "r"(hy[u]), "r"(p2));
                const uint32_t o = atom_xor_shared(a, mz);
                violA |= o & my;
            }
            {   // slot 1: register = high half; register / 32 = bits 21.. of the pair = mulhi(pair, 2048)
                const uint32_t tb = t2 >> 16;
                const uint32_t p2 = __funnelshift_l(0u, B.alive, tb);
                uint32_t wd;
                asm("mul.hi.u32 %0, %1, %2;" : "=r"(wd) : "r"(t2), "r"(B.amask));
                asm("mad.lo.u32 %0, %1, 256, %2;" : "=r"(a) : "r"(wd), "r"(occ_addr + 128u));
                asm("mul.lo.u32 %0, %1, %2;" : "=r"(mz) : "r"(hz[u]), "r"(p2));
                asm("mul.lo.u32 %0, %1, %2;" : "=r"(my) : "r"(hy[u]), "r"(p2));
                const uint32_t o = atom_xor_shared(a, mz);
                violB |= o & my;
            }
        }
    }
}

// One event applied to one candidate's mask word by word: any width, any position (occ = the
// candidate's word 0; its words are 64 apart).
__device__ __noinline__ uint32_t walk_event_general(uint32_t *occ, uint32_t tv, uint32_t width, bool test, bool toggle)
{
    uint32_t viol = 0, left = width, pos = tv;
    while (left) {
        const uint32_t s2 = pos & 31, nn = min(left, 32 - s2);
        const uint32_t m = (nn == 32 ? 0xFFFFFFFFu : ((1u << nn) - 1u)) << s2;
        uint32_t *a = occ + (pos >> 5) * 64;
        const uint32_t o = *a;
        if (test) viol |= o & m;
        if (toggle) *a = o ^ m;
        pos += nn;
        left -= nn;
    }
    return viol;
}

// The 8 events of the group at shared address ga, event by event and word by word: for groups in
// which a walked candidate has an entry with the straddle mark.
__device__ __noinline__ uint2 apply_event_general(uint32_t ga, uint32_t u, uint32_t t2, uint32_t *occA, bool aliveA, bool aliveB)
{
    uint2 viol = make_uint2(0, 0);
    const uint32_t toggle = lds32(ga + 32 + 4 * u), test = lds32(ga + 64 + 4 * u);
    if (!(toggle | test)) return viol;
    const uint32_t wl = (lds32(ga + 96 + 4 * (u >> 1)) >> (16 * (u & 1))) & 0xFFFFu;
    const uint32_t width = (wl & 0x8000u) ? (wl & 0xFFu) : 32u - wl;
    if (aliveA) viol.x = walk_event_general(occA, t2 & 0x7FFFu, width, test != 0, toggle != 0);
    if (aliveB) viol.y = walk_event_general(occA + 32, (t2 >> 16) & 0x7FFFu, width, test != 0, toggle != 0);
    return viol;
}
__device__ __forceinline__ void apply_group_general(uint32_t ga, const uint32_t (&t)[8], uint32_t *occA, bool aliveA, bool aliveB,
                                                    uint32_t &violA, uint32_t &violB)
{
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const uint2 v = apply_event_general(ga, u, t[u], occA, aliveA, aliveB);
        violA |= v.x;
        violB |= v.y;
    }
}

// The ng event groups staged at shared address ev_addr (followed by two more staged groups, which
// are fetched ahead but not applied), applied to the masks of this lane's two candidates.  Table
// entries are fetched two groups ahead of the group that is applied.  With CHECK = false the
// caller vouches that no walked candidate of the warp has a marked entry: the loop body has no
// conditions.  With CHECK = true one vote per group decides between the one-atomic form and the
// general one.
template <bool CHECK>
__device__ __forceinline__ void walk_piece(uint32_t ev_addr, uint32_t ng, const unsigned char *tgb, uint32_t occ_addr,
                                           uint32_t *occA, const WalkSlot &A, const WalkSlot &B, uint32_t &violA,
                                           uint32_t &violB)
{
    const uint32_t marks = (A.alive ? 0x8000u : 0u) | (B.alive ? 0x80000000u : 0u);
    auto apply = [&](uint32_t ga, const uint32_t (&t)[8]) {
        if (CHECK) {
            const uint32_t any = (t[0] | t[1] | t[2] | t[3] | t[4] | t[5] | t[6] | t[7]) & marks;
            if (__any_sync(0xffffffffu, any != 0)) {
                apply_group_general(ga, t, occA, A.alive != 0, B.alive != 0, violA, violB);
                return;
            }
        }
        apply_group(ga, t, occ_addr, A, B, violA, violB);
    };
    uint32_t ta[8], tb[8], tc[8];
    fetch_group(ev_addr, tgb, ta);
    fetch_group(ev_addr + 112, tgb, tb);
    uint32_t g = 0;
    for (; g + 3 <= ng; g += 3) {
        const uint32_t ga = ev_addr + g * 112;
        fetch_group(ga + 224, tgb, tc);
        apply(ga, ta);
        fetch_group(ga + 336, tgb, ta);
        apply(ga + 112, tb);
        fetch_group(ga + 448, tgb, tb);
        apply(ga + 224, tc);
    }
    // up to two groups are left: ta holds group g, tb group g + 1
    if (g < ng) apply(ev_addr + g * 112, ta);
    if (g + 1 < ng) apply(ev_addr + (g + 1) * 112, tb);
}

// The same for programs with vregs wider than a mask word (rare): event by event, word by word,
// nothing fetched ahead.
__device__ __noinline__ void walk_piece_general(const uint4 *s_ev, uint32_t ng, const unsigned char *tgb, uint32_t *occA,
                                                bool aliveA, bool aliveB, uint32_t &violA, uint32_t &violB)
{
    for (uint32_t g = 0; g < ng; ++g) {
        const uint32_t *grp_w = reinterpret_cast<const uint32_t *>(s_ev + (size_t)g * 7);
        const uint16_t *grp_wl = reinterpret_cast<const uint16_t *>(grp_w + 24);
        for (uint32_t u = 0; u < 8; ++u) {
            const uint32_t off = grp_w[u], toggle = grp_w[8 + u], test = grp_w[16 + u], wl = grp_wl[u];
            if (!(toggle | test)) continue;
            const uint32_t width = (wl & 0x8000u) ? (wl & 0xFFu) : 32u - wl;
            const uint32_t t2 = *reinterpret_cast<const uint32_t *>(tgb + off);
            if (aliveA) violA |= walk_event_general(occA, t2 & 0x7FFFu, width, test != 0, toggle != 0);
            if (aliveB) violB |= walk_event_general(occA + 32, (t2 >> 16) & 0x7FFFu, width, test != 0, toggle != 0);
        }
    }
}

// =========================================================================== k_through
// grid (program blocks, groups of 64 candidates): the occupancy of the vregs that stay occupied
// through the whole block (its through-set), for every candidate of the group, as masks in the
// walk's layout [word][slot 0 / 1][lane]; a collision inside the through-set marks the block in the
// candidate's state.  Every chunk walk of the block starts from these masks.
__global__ void __launch_bounds__(256) k_through(const WParams q)
{
    extern __shared__ __align__(16) uint32_t wsm[];
    uint32_t *s_th = wsm;  // [Wp][2][32]
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const uint32_t b = blockIdx.x, grp = blockIdx.y;
    const uint64_t kA = (uint64_t)grp * TGW + 2 * lane, kB = kA + 1;
    uint32_t *csA = q.cstate + kA * 8, *csB = csA + 8;  // rows beyond K exist in the working buffers (whole groups)
    const bool walkedA = kA < q.K && !(csA[CS_WALK] & WALK_FULL), walkedB = kB < q.K && !(csB[CS_WALK] & WALK_FULL);
    const unsigned char *tgb = reinterpret_cast<const unsigned char *>(q.tg + (uint64_t)grp * (q.V + 1) * TGW + 2 * lane);
    for (uint32_t i = threadIdx.x; i < q.Wp * 64; i += blockDim.x) s_th[i] = 0;
    __syncthreads();
    bool thcolA = false, thcolB = false;
    const uint32_t e1 = q.th_off[b + 1];
    for (uint32_t e0 = q.th_off[b] + warp * 8; e0 < e1; e0 += n_warps * 8) {
        uint32_t x[8], t[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) x[u] = e0 + u < e1 ? q.th[e0 + u] : (q.V | (0u << 16));
#pragma unroll
        for (int u = 0; u < 8; ++u) t[u] = *reinterpret_cast<const uint32_t *>(tgb + (size_t)(x[u] & 0xFFFFu) * (TGW * 2));
#pragma unroll
        for (int u = 0; u < 8; ++u) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (!(h ? walkedB : walkedA)) continue;
                uint32_t pos = (h ? (t[u] >> 16) : t[u]) & 0x7FFFu, left = x[u] >> 16;
                while (left) {
                    const uint32_t s2 = pos & 31, n = min(left, 32 - s2);
                    const uint32_t m = (n == 32 ? 0xFFFFFFFFu : ((1u << n) - 1u)) << s2;
                    const uint32_t old = atomicOr(&s_th[((pos >> 5) * 2 + h) * 32 + lane], m);
                    if (h) thcolB |= (old & m) != 0; else thcolA |= (old & m) != 0;
                    pos += n;
                    left -= n;
                }
            }
        }
    }
    if (thcolA) atomicOr(&csA[CS_THCOL], 1u << b);  // through-sets are used only if nB <= 32
    if (thcolB) atomicOr(&csB[CS_THCOL], 1u << b);
    __syncthreads();
    uint32_t *dst = q.thm + ((size_t)grp * q.nB + b) * q.Wp * 64;
    for (uint32_t i = threadIdx.x; i < q.Wp * 64; i += blockDim.x) dst[i] = s_th[i];
}

// =========================================================================== k_walk
// grid (octets of chunks, groups of 64 candidates); one warp per chunk; a lane carries two candidates.
// Shared memory per warp: [occupancy [Wp][2][32]][events of the chunk].
__global__ void __launch_bounds__(WALK_WARPS * 32, 3) k_walk(const WParams q)
{
    extern __shared__ __align__(16) uint32_t wsm[];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const uint32_t per_warp = q.Wp * 64 + ((q.ev_cap >> 3) + 2) * 28;  // words: 112 bytes per group of 8 events
    uint32_t *s_occ = wsm + (size_t)warp * per_warp;             // [Wp][2][32]
    uint4 *s_ev = reinterpret_cast<uint4 *>(s_occ + q.Wp * 64);  // [ev_cap / 8 + 2] groups of 7 x 16 bytes
    const uint32_t grp = blockIdx.y, c = blockIdx.x * n_warps + warp;
    const uint64_t kA = (uint64_t)grp * TGW + 2 * lane, kB = kA + 1;
    uint32_t *csA = q.cstate + kA * 8, *csB = csA + 8;  // rows beyond K exist in the working buffers (whole groups)
    // candidates beyond K, and candidates that are recounted in full anyway (their table may hold
    // anything), are not walked
    const bool walkedA = kA < q.K && !(csA[CS_WALK] & WALK_FULL), walkedB = kB < q.K && !(csB[CS_WALK] & WALK_FULL);
    const unsigned char *tgb = reinterpret_cast<const unsigned char *>(q.tg + (uint64_t)grp * (q.V + 1) * TGW + 2 * lane);
    const uint32_t occ_addr = smem_u32(s_occ) + lane * 4, ev_addr = smem_u32(s_ev);
    WalkSlot A, B;
    A.alive = walkedA ? 1u : 0u; A.amask = walkedA ? 0x7FE0u : 0u;
    B.alive = walkedB ? 1u : 0u; B.amask = walkedB ? 2048u : 0u;
    // no table entry of the group carries the straddle mark: the walk decides nothing per event
    const bool marked = __ldcg(q.grp_flag + grp) != 0;
    if (c < q.nC) {
        // the chunk starts from the through-set masks of its block: made by k_through, or (small jobs,
        // where one launch more costs more than the repeated work) by this warp on the spot
        if (q.use_th && q.thm) {
            const uint32_t *src = q.thm + ((size_t)grp * q.nB + q.chunk_blk[c]) * q.Wp * 64;
            for (uint32_t wd = 0; wd < q.Wp * 2; ++wd) s_occ[wd * 32 + lane] = src[wd * 32 + lane];
        } else {
            for (uint32_t wd = 0; wd < q.Wp * 2; ++wd) s_occ[wd * 32 + lane] = 0;
        }
        if (q.use_th && !q.thm) {
            const uint32_t b = q.chunk_blk[c];
            bool thcolA = false, thcolB = false;
            const uint32_t e1 = q.th_off[b + 1];
            for (uint32_t e0 = q.th_off[b]; e0 < e1; e0 += 8) {  // the table entries of 8 members in flight together
                uint32_t x[8], t[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) x[u] = e0 + u < e1 ? q.th[e0 + u] : (q.V | (0u << 16));
#pragma unroll
                for (int u = 0; u < 8; ++u) t[u] = *reinterpret_cast<const uint32_t *>(tgb + (size_t)(x[u] & 0xFFFFu) * (TGW * 2));
#pragma unroll
                for (int u = 0; u < 8; ++u) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (!(h ? walkedB : walkedA)) continue;
                        uint32_t pos = (h ? (t[u] >> 16) : t[u]) & 0x7FFFu, left = x[u] >> 16;
                        while (left) {
                            const uint32_t s2 = pos & 31, n = min(left, 32 - s2);
                            const uint32_t m = (n == 32 ? 0xFFFFFFFFu : ((1u << n) - 1u)) << s2;
                            uint32_t *a = &s_occ[((pos >> 5) * 2 + h) * 32 + lane];
                            const uint32_t old = *a;
                            *a = old | m;
                            if (h) thcolB |= (old & m) != 0; else thcolA |= (old & m) != 0;
                            pos += n;
                            left -= n;
                        }
                    }
                }
            }
            if (thcolA) atomicOr(&csA[CS_THCOL], 1u << b);  // through-sets are used only if nB <= 32
            if (thcolB) atomicOr(&csB[CS_THCOL], 1u << b);
        }
        uint32_t violA = 0, violB = 0;
        const uint32_t s0 = q.cev_off[c], n_ev = q.cev_off[c + 1] - s0;  // a multiple of 8 events
        for (uint32_t done = 0; done < n_ev; done += q.ev_cap) {
            const uint32_t n = min(q.ev_cap, n_ev - done), ng = n >> 3;
            __syncwarp();
            {   // events of this piece and of the two groups after it (the event array ends with two
                // no-op groups), once: 7 x 16 bytes per group of 8
                const uint4 *src = q.ev + (size_t)((s0 + done) >> 3) * 7;
                for (uint32_t i = lane; i < (ng + 2) * 7; i += 32) s_ev[i] = src[i];
            }
            __syncwarp();
            if (q.wmax > 32) walk_piece_general(s_ev, ng, tgb, s_occ + lane, walkedA, walkedB, violA, violB);
            else if (marked) walk_piece<true>(ev_addr, ng, tgb, occ_addr, s_occ + lane, A, B, violA, violB);
            else walk_piece<false>(ev_addr, ng, tgb, occ_addr, s_occ + lane, A, B, violA, violB);
        }
        if (violA && walkedA) {
            atomicOr(&q.anom[kA * q.AW + (c >> 5)], 1u << (c & 31));
            atomicOr(&csA[CS_WALK], WALK_ANOM);
        }
        if (violB && walkedB) {
            atomicOr(&q.anom[kB * q.AW + (c >> 5)], 1u << (c & 31));
            atomicOr(&csB[CS_WALK], WALK_ANOM);
        }
    }
    // the thread block that finishes a group's last chunk writes the verdicts of the group's clean
    // candidates and lists the others for the recount
    __shared__ uint32_t s_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(&q.grp_done[grp], 1u) == gridDim.x - 1 ? 1u : 0u;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (threadIdx.x == 0) q.grp_flag[grp] = 0;  // every block of the group has read it: clear for the next pass
    for (uint32_t j = warp; j < TGW; j += n_warps) {
        const uint64_t kk = (uint64_t)grp * TGW + j;
        if (kk < q.K) finish_candidate(kk, q.nC, q.AW, q.list_all, q.cstate, q.anom, q.chunk_blk, q.work, q.racc, q.out);
    }
}

// =========================================================================== verdicts / work list
// Verdicts of the candidates the walk vouches for.  For the others, work items for k_recount:
// every chunk that needs an exact recount is cut into RC_PARTS pieces, the general bank tally into
// RC_BANK_PARTS slices, and every block whose through-set collided gets one item for the
// definitions the walk skipped in its other chunks; racc[k][3] counts the items pending.  An item
// is (candidate, code) with code = kind << 30 | piece << 24 | chunk (or block).
#define RC_PARTS 2
#define RC_HDR 4  // words in front of the work items: item count, cursor of the first round, cursor of the second
#define RC_BANK_PARTS 4
#define RC_KIND_ALL 0u     // every definition of the piece
#define RC_KIND_THROUGH 1u // a block whose through-set collided: the definitions the walk skipped, chunk = block
#define RC_KIND_BANK 2u
__device__ __forceinline__ uint32_t rc_code(uint32_t kind, uint32_t piece, uint32_t chunk)
{
    return (kind << 30) | (piece << 24) | chunk;
}

// One warp finishes candidate k: the verdict if nothing is left to recount, else its work items.
// cstate / anom words that other thread blocks updated with atomics are read from L2.
__device__ void finish_candidate(uint64_t k, uint32_t nC, uint32_t AW, int list_all, const uint32_t *cstate,
                                 const uint32_t *anom, const uint32_t *__restrict__ chunk_blk, uint32_t *work,
                                 uint32_t *racc, vl_verdict *out)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t *cs = cstate + k * 8;
    const uint32_t walk = __ldcg(cs + CS_WALK), thcol = __ldcg(cs + CS_THCOL);
    if (!list_all && !(walk | thcol)) {
        if (lane == 0) {
            const uint32_t fl = __ldcg(cs + CS_FLAGS), first = __ldcg(cs + CS_FIRST);
            vl_verdict vd;
            vd.flags = fl ? fl : (uint32_t)VL_PASS;
            vd.first_violation_instr = first == 0xFFFFFFFFu ? -1 : (int32_t)first;
            vd.conflict_pairs = 0;
            vd.bank_conflicts = __ldcg(cs + CS_BANK);
            out[k] = vd;
        }
        return;
    }
    // a chunk that collided (or a candidate with several out-of-file vregs): every definition;
    // a block whose through-set collided: the definitions the walk skipped in its other chunks (a
    // vreg redefined from itself while it stays occupied), since everything else in them was walked
    // exactly
    const bool full = walk & WALK_FULL;
    auto all_defs = [&](uint32_t c) -> bool {
        return c < nC && (full || ((__ldcg(anom + k * AW + (c >> 5)) >> (c & 31)) & 1u));
    };
    uint32_t n_chunks = 0;
    for (uint32_t c0 = 0; c0 < nC; c0 += 32) n_chunks += __popc(__ballot_sync(0xffffffffu, all_defs(c0 + lane)));
    const uint32_t n_blocks = full ? 0u : __popc(thcol);
    // the fast-path tally is one item per candidate (its table column is fetched once); the general tally
    // of the other programs, which every candidate takes, is sliced
    const uint32_t n_bank = list_all ? (uint32_t)RC_BANK_PARTS : 1u;
    const uint32_t n = n_bank + RC_PARTS * n_chunks + n_blocks;
    uint32_t at = 0;
    if (lane == 0) {
        racc[k * 4 + 3] = n;
        at = atomicAdd(work, n);
    }
    at = __shfl_sync(0xffffffffu, at, 0);
    if (lane < n_bank) {
        work[RC_HDR + 2 * (at + lane)] = (uint32_t)k;
        work[RC_HDR + 1 + 2 * (at + lane)] = rc_code(RC_KIND_BANK, lane, 0);
    }
    at += n_bank;
    if (!full && ((thcol >> lane) & 1u)) {  // through-sets are used only if the program has at most 32 blocks
        const uint32_t slot = at + __popc(thcol & ((1u << lane) - 1u));
        work[RC_HDR + 2 * slot] = (uint32_t)k;
        work[RC_HDR + 1 + 2 * slot] = rc_code(RC_KIND_THROUGH, 0, lane);
    }
    at += n_blocks;
    for (uint32_t c0 = 0; c0 < nC; c0 += 32) {
        const bool kd = all_defs(c0 + lane);
        const uint32_t m = __ballot_sync(0xffffffffu, kd);
        if (kd) {
            const uint32_t slot = at + RC_PARTS * __popc(m & ((1u << lane) - 1u));
#pragma unroll
            for (uint32_t part = 0; part < RC_PARTS; ++part) {
                work[RC_HDR + 2 * (slot + part)] = (uint32_t)k;
                work[RC_HDR + 1 + 2 * (slot + part)] = rc_code(RC_KIND_ALL, part, c0 + lane);
            }
        }
        at += RC_PARTS * __popc(m);
    }
}

// Stand-alone form for programs without walk items (no instructions): one warp per candidate.
__global__ void k_finish(uint64_t K, uint32_t nC, uint32_t AW, int list_all, const uint32_t *cstate,
                         const uint32_t *anom, const uint32_t *__restrict__ chunk_blk, uint32_t *work, uint32_t *racc,
                         vl_verdict *out)
{
    const uint64_t k = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (k < K) finish_candidate(k, nC, AW, list_all, cstate, anom, chunk_blk, work, racc, out);
}

// Bank list entries [e_lo, e_hi) with N distinct source vregs each: how many sources hold the register
// of an earlier source of the same entry.  regs[v] = register of vreg v (shared memory).  8 entries per
// thread and round; the entries of the next round are fetched meanwhile.
template <int N>
__device__ __forceinline__ uint32_t bank_duplicates(const uint2 *__restrict__ list, uint32_t e_lo, uint32_t e_hi,
                                                    const uint32_t *regs, uint32_t tid)
{
    uint32_t dups = 0;
    uint2 id_next[8];
#pragma unroll
    for (int u = 0; u < 8; ++u)
        id_next[u] = e_lo + tid + u * RC_THREADS < e_hi ? list[e_lo + tid + u * RC_THREADS] : make_uint2(0, 0);
    for (uint32_t e0 = e_lo + tid; e0 < e_hi; e0 += 8 * RC_THREADS) {
        uint2 idv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            idv[u] = id_next[u];
            const uint32_t en = e0 + (8 + u) * RC_THREADS;
            id_next[u] = en < e_hi ? list[en] : make_uint2(0, 0);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (e0 + u * RC_THREADS >= e_hi) break;
            const uint32_t x0 = regs[idv[u].x & 0xFFFFu], x1 = regs[idv[u].x >> 16];
            dups += (x1 == x0);
            if (N >= 3) {
                const uint32_t x2 = regs[idv[u].y & 0xFFFFu];
                dups += (x2 == x0) | (x2 == x1);
                if (N >= 4) {
                    const uint32_t x3 = regs[idv[u].y >> 16];
                    dups += (x3 == x0) | (x3 == x1) | (x3 == x2);
                }
            }
        }
    }
    return dups;
}

// =========================================================================== k_recount
// Exact answers for the listed work items; thread blocks loop over the list.  A chunk item recounts
// the overlaps of one piece of a chunk from the live-after lists (the warps share the piece's
// instructions; the lanes of a warp fetch the bookkeeping of 32 instructions at a time); a bank
// item does a slice of the general bank tally (distinct registers rather than distinct vregs).
// The candidate's register and the width of a vreg are fetched from global memory the first time
// an item needs them and kept in a shared-memory cache (CACHE; one word per vreg, valid bit 31):
// the live-after sets of neighbouring instructions are nearly the same, so a piece touches a few
// hundred vregs, not the whole table column.  Results are added to the candidate's accumulators;
// the item that finishes last writes the verdict.
template <bool CACHE>
__global__ void __launch_bounds__(RC_THREADS) k_recount(const RParams q)
{
    extern __shared__ __align__(16) uint32_t Cv[];  // [V] register | width << 16 | valid << 31
    __shared__ uint32_t s_pairs, s_mind, s_bank, s_big;
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr uint32_t NW = RC_THREADS / 32;
    const uint32_t nitems = q.work[0];
    __shared__ uint32_t s_item;
    // The items differ a lot in length: thread blocks take the next one from a shared cursor.  Two rounds
    // over the list: the long items first (a bank tally sweeps the whole program, a through-set item is
    // quadratic in the set), then the chunk pieces, so that no long item starts when the others end.
    for (uint32_t round = 0; round < 2;) {
        __syncthreads();
        if (tid == 0) s_item = atomicAdd(q.work + 1 + round, 1u);
        __syncthreads();
        const uint32_t it = s_item;
        if (it >= nitems) { ++round; continue; }
        const uint64_t k = q.work[RC_HDR + 2 * it];
        const uint32_t code = q.work[RC_HDR + 1 + 2 * it];
        const uint32_t kind = code >> 30, part = (code >> 24) & 63u, c = code & 0xFFFFFFu;
        if ((kind == RC_KIND_ALL) != (round == 1)) continue;
        const uint32_t *cs = q.cstate + k * 8;
        const uint16_t *tg = q.tg + (k / TGW) * (uint64_t)(q.V + 1) * TGW + (k & (TGW - 1));
        // a single out-of-file vreg sits parked in the table: its true register is in the candidate's state
        const uint32_t out_v = cs[CS_NOUT] == 1 ? cs[CS_OUTV] : 0xFFFFFFFFu, out_raw = cs[CS_OUTRAW];
        // a candidate with several out-of-file vregs was not walked and keeps its table unmarked
        const uint32_t tmask = (cs[CS_WALK] & WALK_FULL) ? 0xFFFFu : 0x7FFFu;
        __syncthreads();
        if (CACHE)
            for (uint32_t v = tid; v < q.V; v += RC_THREADS) Cv[v] = 0;
        if (tid == 0) { s_pairs = 0; s_mind = 0xFFFFFFFFu; s_bank = 0; }
        __syncthreads();
        // register (low 16 bits) and width (bits 16..23) of vreg v for this candidate
        auto fetch = [&](uint32_t v) -> uint32_t {
            const uint32_t r = v == out_v ? out_raw : ((uint32_t)tg[(size_t)v * TGW] & tmask);
            return r | ((q.vinfo[v] & 0xFFu) << 16);
        };
        auto reg_w = [&](uint32_t v) -> uint32_t {
            if (!CACHE) return fetch(v);
            uint32_t x = Cv[v];
            if (!(x >> 31)) {
                x = fetch(v) | 0x80000000u;
                Cv[v] = x;  // several threads may store the same word
            }
            return x;
        };
        if (kind == RC_KIND_THROUGH) {
            // The through-set of block c collided.  In a chunk of the block whose own walk was clean,
            // everything else that is live is disjoint from the through-set and from each other, so a
            // skipped definition of a through-set vreg overlaps exactly the through-set members that
            // overlap it, whatever the instruction: count those once per member, then add them up over
            // the skipped definitions.  (Chunks that did collide are recounted in full by their own items.)
            const uint32_t t0 = q.th_off[c], n_th = q.th_off[c + 1] - t0;
            uint32_t *ids = Cv;  // [n_th] member vreg ids (ascending), [n_th] register | width << 16, [n_th] counts
            uint32_t *mem = Cv + n_th, *cnt_th = Cv + 2 * n_th;
            const bool fits = CACHE && 3 * n_th <= q.V;
            if (fits) {
                __syncthreads();
                for (uint32_t j = tid; j < n_th; j += RC_THREADS) {
                    const uint32_t v = q.th[t0 + j] & 0xFFFFu;
                    ids[j] = v;
                    mem[j] = fetch(v);
                }
                __syncthreads();
                for (uint32_t j = tid; j < n_th; j += RC_THREADS) {
                    const uint32_t s = mem[j] & 0xFFFFu, w = (mem[j] >> 16) & 0xFFu;
                    uint32_t cc = 0;
                    for (uint32_t u = 0; u < n_th; ++u)
                        if (u != j && ranges_overlap(s, w, mem[u] & 0xFFFFu, (mem[u] >> 16) & 0xFFu)) ++cc;
                    cnt_th[j] = cc;
                }
                __syncthreads();
            }
            // overlap count of through-set member v (0 if v is not a member): the list is ascending
            auto count_of = [&](uint32_t v) -> uint32_t {
                uint32_t lo_j = 0, hi_j = n_th;
                while (lo_j < hi_j) {
                    const uint32_t mid = (lo_j + hi_j) >> 1;
                    if ((fits ? ids[mid] : (q.th[t0 + mid] & 0xFFFFu)) < v) lo_j = mid + 1; else hi_j = mid;
                }
                if (lo_j >= n_th || (fits ? ids[lo_j] : (q.th[t0 + lo_j] & 0xFFFFu)) != v) return 0u;
                if (fits) return cnt_th[lo_j];
                const uint32_t x = fetch(v);
                uint32_t cc = 0;
                for (uint32_t u = 0; u < n_th; ++u) {
                    if (u == lo_j) continue;
                    const uint32_t y = fetch(q.th[t0 + u] & 0xFFFFu);
                    if (ranges_overlap(x & 0xFFFFu, (x >> 16) & 0xFFu, y & 0xFFFFu, (y >> 16) & 0xFFu)) ++cc;
                }
                return cc;
            };
            // the program's skipped definitions are listed as {instruction, chunk, vreg, block}
            uint32_t pairs = 0, mind = 0xFFFFFFFFu;
            const uint32_t n_el = *q.el_count;
            for (uint32_t e = tid; e < n_el; e += RC_THREADS) {
                const uint4 x = q.el[e];
                if (x.w != c) continue;
                if ((q.anom[k * q.AW + (x.y >> 5)] >> (x.y & 31)) & 1u) continue;
                const uint32_t cn = count_of(x.z);
                if (cn) { pairs += cn; mind = min(mind, x.x); }
            }
#pragma unroll
            for (int dd = 16; dd; dd >>= 1) {
                pairs += __shfl_xor_sync(0xffffffffu, pairs, dd);
                mind = min(mind, __shfl_xor_sync(0xffffffffu, mind, dd));
            }
            if (lane == 0 && pairs) {
                atomicAdd(&s_pairs, pairs);
                atomicMin(&s_mind, mind);
            }
        } else if (kind != RC_KIND_BANK) {
            const uint32_t ci0 = q.chunk_i0[c], cn = q.chunk_i1[c] - ci0;
            const uint32_t i_lo = ci0 + (uint32_t)((uint64_t)cn * part / RC_PARTS);
            const uint32_t i_hi = ci0 + (uint32_t)((uint64_t)cn * (part + 1) / RC_PARTS);
            uint32_t pairs = 0, mind = 0xFFFFFFFFu;
            // The vregs that stay occupied through the whole block (its through-set) are live after every
            // instruction of it.  Rather than meeting them again in every live-after list, the block
            // counts them once into two arrays over the registers (cover[r]: members whose range holds r,
            // start[r]: members whose range starts at r); a definition with range [s, s+w) then overlaps
            // cover[s] + start[s+1] + ... + start[s+w-1] of them, and only the short list (live after,
            // not in the through-set) is scanned entry by entry.  Needs every member inside the arrays
            // (R registers: the file plus the widest vreg); otherwise the full lists are scanned.
            const uint32_t blk = q.chunk_blk[c];
            const uint32_t t0 = q.th_off[blk], n_th = q.th_off[blk + 1] - t0;
            const uint32_t ls_sub = q.ls_adj[blk], ls_mul = q.th_cnt[blk];
            uint32_t *cover = Cv + q.V + 4, *start = cover + q.R;
            bool use_short = CACHE && n_th > 0 && ls_mul == n_th;
            if (use_short) {
                for (uint32_t r = tid; r < 2 * q.R; r += RC_THREADS) cover[r] = 0;
                if (tid == 0) s_big = 0;
                __syncthreads();
                for (uint32_t j = tid; j < n_th; j += RC_THREADS) {
                    const uint32_t v = q.th[t0 + j] & 0xFFFFu;
                    const uint32_t f = fetch(v), reg = f & 0xFFFFu, w = (f >> 16) & 0xFFu;
                    Cv[v] = f | 0xC0000000u;  // valid, member of the through-set
                    if (reg + w <= q.R) {
                        atomicAdd(&start[reg], 1u);
                        for (uint32_t r = reg; r < reg + w; ++r) atomicAdd(&cover[r], 1u);
                    } else {
                        s_big = 1;
                    }
                }
                __syncthreads();
                use_short = s_big == 0;
            }
            const uint32_t *lst = use_short ? q.ls : q.lo;
            // first entry and length of instruction i's list, from its two live-after offsets
            auto list_lo = [&](uint32_t i, uint32_t off_i) { return use_short ? off_i - ls_sub - i * ls_mul : off_i; };
            auto list_n = [&](uint32_t off_i, uint32_t off_i1) { return off_i1 - off_i - (use_short ? ls_mul : 0u); };
            if (CACHE && i_lo < i_hi) {
                // Every vreg that is live after an instruction of the piece is live after its first
                // instruction or defined inside the piece: the whole block fetches those into the cache in
                // one go, so that the instruction-by-instruction recount below finds them there instead of
                // waiting for global memory once per instruction.
                const uint32_t f0 = q.lo_off[i_lo], f1 = q.lo_off[i_lo + 1];
                const uint32_t l0 = list_lo(i_lo, f0), l1 = l0 + list_n(f0, f1);
                for (uint32_t e = l0 + tid; e < l1; e += RC_THREADS) {
                    const uint32_t v = lst[e];
                    if (!(Cv[v] >> 31)) Cv[v] = fetch(v) | 0x80000000u;
                }
                for (uint32_t i = i_lo + tid; i < i_hi; i += RC_THREADS) {
                    const uint32_t o0 = q.op_off[i], nd = q.ndefs[i];
                    for (uint32_t d = o0; d < o0 + nd; ++d) {
                        const uint32_t v = q.op_vreg[d];
                        if (!(Cv[v] >> 31)) Cv[v] = fetch(v) | 0x80000000u;
                    }
                }
                __syncthreads();
            }
            if (use_short) {
                // Short lists (the through-set is counted from the arrays): two lanes per instruction, 128
                // instructions per round, so that the loads of a whole round (bookkeeping, then defined vregs
                // and list entries) are in flight together instead of instruction after instruction.
                const uint32_t sub = lane & 1u, slot = tid >> 1;
                for (uint32_t ib = i_lo; ib < i_hi; ib += RC_THREADS / 2) {
                    const uint32_t i = ib + slot;
                    uint32_t cnt_i = 0;
                    if (i < i_hi) {
                        const uint32_t o0 = q.op_off[i], nd = q.ndefs[i];
                        const uint32_t f0 = q.lo_off[i], f1 = q.lo_off[i + 1];
                        const uint32_t l0 = list_lo(i, f0), l1 = l0 + list_n(f0, f1);
                        for (uint32_t d = o0; d < o0 + nd; ++d) {
                            const uint32_t v = q.op_vreg[d];
                            const uint32_t sw = reg_w(v);
                            const uint32_t s = sw & 0xFFFFu, w = (sw >> 16) & 0xFFu;
                            uint32_t cnt = 0;
                            if (s < q.R) {  // the through-set members that overlap [s, s+w), v itself excepted
                                if (sub == 0) cnt = cover[s] - ((sw >> 30) & 1u);
                                for (uint32_t r = s + 1 + sub; r < min(s + w, q.R); r += 2) cnt += start[r];
                            }
                            for (uint32_t e0 = l0 + sub; e0 < l1; e0 += 16) {  // 8 list entries per lane in flight
                                uint32_t us[8], xs[8];
#pragma unroll
                                for (int u = 0; u < 8; ++u) {
                                    const uint32_t e = e0 + u * 2;
                                    us[u] = e < l1 ? lst[e] : v;
                                }
#pragma unroll
                                for (int u = 0; u < 8; ++u) xs[u] = reg_w(us[u]);
#pragma unroll
                                for (int u = 0; u < 8; ++u)
                                    if (us[u] != v && ranges_overlap(s, w, xs[u] & 0xFFFFu, (xs[u] >> 16) & 0xFFu)) ++cnt;
                            }
                            // co-defined vregs that are not live after the instruction
                            if (nd > 1)
                                for (uint32_t d2 = o0 + sub; d2 < o0 + nd; d2 += 2) {
                                    if (d2 == d || !(q.opflags[d2] & OPF_DEAD)) continue;
                                    const uint32_t x = reg_w(q.op_vreg[d2]);
                                    if (ranges_overlap(s, w, x & 0xFFFFu, (x >> 16) & 0xFFu)) ++cnt;
                                }
                            cnt_i += cnt;
                        }
                    }
                    cnt_i += __shfl_xor_sync(0xffffffffu, cnt_i, 1);
                    if (cnt_i && sub == 0) { pairs += cnt_i; mind = min(mind, i); }
                }
#pragma unroll
                for (int dd = 16; dd; dd >>= 1) {  // (lane 0 reports for the warp)
                    pairs += __shfl_xor_sync(0xffffffffu, pairs, dd);
                    mind = min(mind, __shfl_xor_sync(0xffffffffu, mind, dd));
                }
            }
            // full lists: this warp's instructions are i_lo + warp, i_lo + warp + NW, ...; 32 of them per round
            for (uint32_t ib = i_lo + warp; !use_short && ib < i_hi; ib += 32 * NW) {
                const uint32_t my_i = ib + lane * NW;
                uint32_t m_o0 = 0, m_nd = 0, m_l0 = 0, m_l1 = 0;
                if (my_i < i_hi) {
                    m_o0 = q.op_off[my_i]; m_nd = q.ndefs[my_i];
                    const uint32_t f0 = q.lo_off[my_i], f1 = q.lo_off[my_i + 1];
                    m_l0 = list_lo(my_i, f0);
                    m_l1 = m_l0 + list_n(f0, f1);
                }
                // first defined vreg of each instruction, fetched by the lane that holds its bookkeeping
                uint32_t m_v0 = 0;
                if (m_nd) m_v0 = q.op_vreg[m_o0];
                uint32_t todo = __ballot_sync(0xffffffffu, m_nd != 0);
                // the first 256 entries of the next instruction's list are fetched while the current
                // instruction is recounted
                uint32_t us_nx[8];
                auto fetch_list = [&](int src) {
                    const uint32_t l0 = __shfl_sync(0xffffffffu, m_l0, src), l1 = __shfl_sync(0xffffffffu, m_l1, src);
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const uint32_t e = l0 + u * 32 + lane;
                        us_nx[u] = e < l1 ? lst[e] : 0xFFFFFFFFu;
                    }
                };
                if (todo) fetch_list(__ffs(todo) - 1);
                while (todo) {
                    const int src = __ffs(todo) - 1;
                    todo &= todo - 1;
                    uint32_t us0[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) us0[u] = us_nx[u];
                    if (todo) fetch_list(__ffs(todo) - 1);
                    const uint32_t i = ib + (uint32_t)src * NW;
                    const uint32_t o0 = __shfl_sync(0xffffffffu, m_o0, src), nd = __shfl_sync(0xffffffffu, m_nd, src);
                    const uint32_t l0 = __shfl_sync(0xffffffffu, m_l0, src), l1 = __shfl_sync(0xffffffffu, m_l1, src);
                    const uint32_t v0 = __shfl_sync(0xffffffffu, m_v0, src);
                    for (uint32_t d = o0; d < o0 + nd; ++d) {
                        const uint32_t v = d == o0 ? v0 : q.op_vreg[d];
                        const uint32_t sw = reg_w(v);
                        const uint32_t s = sw & 0xFFFFu, w = (sw >> 16) & 0xFFu;
                        uint32_t cnt = 0;
                        if (use_short && s < q.R) {  // the through-set members that overlap [s, s+w), v itself excepted
                            if (lane == 0) cnt = cover[s] - ((sw >> 30) & 1u);
                            for (uint32_t r = s + 1 + lane; r < min(s + w, q.R); r += 32) cnt += start[r];
                        }
                        for (uint32_t e0 = l0; e0 < l1; e0 += 256) {  // 8 list entries per lane in flight
                            uint32_t us[8], xs[8];
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                const uint32_t e = e0 + u * 32 + lane;
                                us[u] = e0 == l0 ? us0[u] : (e < l1 ? lst[e] : 0xFFFFFFFFu);
                                if (us[u] == 0xFFFFFFFFu) us[u] = v;
                            }
                            // (with the cache, every entry of the list and v itself were fetched up front)
#pragma unroll
                            for (int u = 0; u < 8; ++u) xs[u] = CACHE ? Cv[us[u]] : fetch(us[u]);
#pragma unroll
                            for (int u = 0; u < 8; ++u)
                                if (us[u] != v && ranges_overlap(s, w, xs[u] & 0xFFFFu, (xs[u] >> 16) & 0xFFu)) ++cnt;
                        }
                        // co-defined vregs that are not live after the instruction
                        if (nd > 1)
                            for (uint32_t d2 = o0 + lane; d2 < o0 + nd; d2 += 32) {
                                if (d2 == d || !(q.opflags[d2] & OPF_DEAD)) continue;
                                const uint32_t x = reg_w(q.op_vreg[d2]);
                                if (ranges_overlap(s, w, x & 0xFFFFu, (x >> 16) & 0xFFu)) ++cnt;
                            }
#pragma unroll
                        for (int dd = 16; dd; dd >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, dd);
                        if (cnt) { pairs += cnt; mind = min(mind, i); }
                    }
                }
            }
            if (lane == 0 && pairs) {
                atomicAdd(&s_pairs, pairs);
                atomicMin(&s_mind, mind);
            }
        } else {
            // a source counts when its register is new among the instruction's sources and its bank is not
            uint32_t bt = 0;
            if (CACHE && q.bank_fast) {
                // The table kernel's tally (sources minus banks touched, per instruction) counts a register
                // that two source vregs share twice: the exact tally is that figure minus the number of such
                // duplicates.  The candidate's registers are fetched in one go (every load in flight at once),
                // then the list is swept from shared memory, one segment per source count.
#pragma unroll 8
                for (uint32_t v = tid; v < q.V; v += RC_THREADS)
                    Cv[v] = v == out_v ? out_raw : ((uint32_t)tg[(size_t)v * TGW] & tmask);
                __syncthreads();
                const uint32_t dups = bank_duplicates<2>(q.bank_list, q.bank_seg[0], q.bank_seg[1], Cv, tid) +
                                      bank_duplicates<3>(q.bank_list, q.bank_seg[1], q.bank_seg[2], Cv, tid) +
                                      bank_duplicates<4>(q.bank_list, q.bank_seg[2], q.bank_seg[3], Cv, tid);
                if (tid == 0) atomicAdd(&s_bank, cs[CS_BANK]);
                if (dups) atomicSub(&s_bank, dups);
            } else
            if (q.bank_fast) {
                const uint32_t n_all = q.bank_seg[3];
                const uint32_t e_lo = 0, e_hi = n_all;  // (one item per candidate: part is 0)
                // 8 list entries per thread and round; the entries of the next round are fetched meanwhile
                uint2 id_next[8];
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    id_next[u] = e_lo + tid + u * RC_THREADS < e_hi ? q.bank_list[e_lo + tid + u * RC_THREADS] : make_uint2(0, 0);
                for (uint32_t e0 = e_lo + tid; e0 < e_hi; e0 += 8 * RC_THREADS) {
                    uint2 idv[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        idv[u] = id_next[u];
                        const uint32_t en = e0 + (8 + u) * RC_THREADS;
                        id_next[u] = en < e_hi ? q.bank_list[en] : make_uint2(0, 0);
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const uint32_t e = e0 + u * RC_THREADS;
                        if (e >= e_hi) break;
                        const uint2 ids = idv[u];
                        const uint32_t n = e < q.bank_seg[1] ? 2u : (e < q.bank_seg[2] ? 3u : 4u);
                        uint32_t x[4];
                        x[0] = reg_w(ids.x & 0xFFFFu) & 0xFFFFu; x[1] = reg_w(ids.x >> 16) & 0xFFFFu;
                        x[2] = reg_w(ids.y & 0xFFFFu) & 0xFFFFu; x[3] = reg_w(ids.y >> 16) & 0xFFFFu;
#pragma unroll
                        for (uint32_t a = 1; a < 4; ++a) {
                            if (a >= n) break;
                            bool seen_value = false, seen_bank = false;
#pragma unroll
                            for (uint32_t bb = 0; bb < a; ++bb) {
                                seen_value |= (x[bb] == x[a]);
                                seen_bank |= ((x[bb] ^ x[a]) & (q.B - 1)) == 0;
                            }
                            if (!seen_value && seen_bank) ++bt;
                        }
                    }
                }
            } else {
                const uint32_t i_lo = (uint32_t)((uint64_t)q.nI * part / RC_BANK_PARTS);
                const uint32_t i_hi = (uint32_t)((uint64_t)q.nI * (part + 1) / RC_BANK_PARTS);
                for (uint32_t i = i_lo + tid; i < i_hi; i += RC_THREADS) {
                    const uint32_t u0 = q.op_off[i] + q.ndefs[i], u1 = q.op_off[i + 1];
                    for (uint32_t a = u0 + 1; a < u1; ++a) {
                        const uint32_t xa = reg_w(q.op_vreg[a]) & 0xFFFFu;
                        bool seen_value = false, seen_bank = false;
                        for (uint32_t bb = u0; bb < a; ++bb) {
                            const uint32_t xb = reg_w(q.op_vreg[bb]) & 0xFFFFu;
                            seen_value |= (xb == xa);
                            seen_bank |= (xb % q.B == xa % q.B);
                        }
                        if (!seen_value && seen_bank) ++bt;
                    }
                }
            }
#pragma unroll
            for (int d = 16; d; d >>= 1) bt += __shfl_xor_sync(0xffffffffu, bt, d);
            if (lane == 0 && bt) atomicAdd(&s_bank, bt);
        }
        __syncthreads();
        if (tid == 0) {
            uint32_t *acc = q.racc + k * 4;
            if (s_pairs) atomicAdd(&acc[0], s_pairs);
            if (s_mind != 0xFFFFFFFFu) atomicMax(&acc[1], ~s_mind);  // accumulators start at 0: keep the complement
            if (s_bank) atomicAdd(&acc[2], s_bank);
            __threadfence();
            if (atomicSub(&acc[3], 1u) == 1u) {  // last item of this candidate
                __threadfence();
                const uint32_t pairs = atomicAdd(&acc[0], 0u), mind = ~atomicMax(&acc[1], 0u),
                               bank = atomicAdd(&acc[2], 0u);
                uint32_t flags = cs[CS_FLAGS] | (pairs ? (uint32_t)VL_INTERFERENCE : 0u);
                if (!flags) flags = VL_PASS;
                const uint32_t first = min(cs[CS_FIRST], mind);
                vl_verdict vd;
                vd.flags = flags;
                vd.first_violation_instr = first == 0xFFFFFFFFu ? -1 : (int32_t)first;
                vd.conflict_pairs = pairs;
                vd.bank_conflicts = bank;
                q.out[k] = vd;
            }
        }
    }
}

// --------------------------------------------------------------------------- host
namespace {
struct Plan { uint32_t G, NT, NS, smem, off_region, off_misc, off_tail; bool ok; };  // G = 8: the eight-candidate kernel

inline uint64_t align16(uint64_t x) { return (x + 15u) & ~15ull; }

// Shared memory of one k_tables block: [T][copy ring][misc].
Plan make_plan(const vl_program *p, uint32_t G, uint32_t NT, uint32_t budget)
{
    Plan pl{};
    pl.G = G; pl.NT = NT;
    const uint64_t stage = (uint64_t)NT * 8 * 2 * G;
    const uint64_t tbytes = align16((uint64_t)(p->V + 1) * G * 2);
    const uint64_t misc = align16(sizeof(TMisc));
    const uint64_t hbytes = align16((uint64_t)(p->V + 1) * 2);  // the bank nibbles reuse the copy ring
    pl.ok = false;
    if (tbytes + misc + std::max(2 * stage, hbytes) > budget) return pl;
    pl.NS = (uint32_t)std::min<uint64_t>(MAX_STAGES, (budget - tbytes - misc) / stage);
    pl.off_region = (uint32_t)tbytes;
    pl.off_misc = (uint32_t)(tbytes + std::max(pl.NS * stage, hbytes));
    pl.smem = pl.off_misc + (uint32_t)misc;
    pl.ok = true;
    return pl;
}

// Shared memory of one k_tables8 block: [T, 16 bytes per vreg][copy ring][tail buffer][misc]; the
// bank nibbles (4 bytes per vreg) reuse the copy ring.
Plan make_plan8(const vl_program *p, uint32_t NT, uint32_t budget)
{
    Plan pl{};
    pl.G = 8; pl.NT = NT;
    const uint64_t stage = (uint64_t)NT * 4 * 2 * 8;
    const uint64_t tbytes = ((uint64_t)(p->V + 1) * 16 + 127) & ~127ull;  // the ring is the target of tiled copies
    const uint64_t tail = 8 * 512;
    const uint64_t misc = align16(sizeof(TMisc));
    const uint64_t hbytes = ((uint64_t)(p->V + 1) * 4 + 127) & ~127ull;
    pl.ok = false;
    if (tbytes + tail + misc + std::max(2 * stage, hbytes) > budget) return pl;
    pl.NS = (uint32_t)std::min<uint64_t>(MAX_STAGES, (budget - tbytes - tail - misc) / stage);
    pl.off_region = (uint32_t)tbytes;
    pl.off_tail = (uint32_t)(tbytes + std::max(pl.NS * stage, hbytes));
    pl.off_misc = pl.off_tail + (uint32_t)tail;
    pl.smem = pl.off_misc + (uint32_t)misc;
    pl.ok = true;
    return pl;
}

// The candidate rows of one pass as a 3-D tensor for the tiled copies of k_tables8:
// [n rows][nfull chunks][256 operands], a box = 8 rows x (tile / 256) chunks x 256 operands.
typedef CUresult (*tm_encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                 const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled, asked from the runtime once per process.
int tensor_encoder(vl_program *p, tm_encode_fn *out)
{
    static std::mutex mtx;
    static tm_encode_fn encode = nullptr;
    std::lock_guard<std::mutex> lock(mtx);
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
            p->last_cuda_error = (int)(e != cudaSuccess ? e : cudaErrorUnknown);
            return VL_ERR_CUDA;
        }
        encode = (tm_encode_fn)fn;
    }
    *out = encode;
    return VL_OK;
}

int encode_row_tensor(vl_program *p, CUtensorMap *tm, const uint16_t *d_cand, uint64_t n, uint64_t pitch, uint32_t nfull,
                      uint32_t chunks_per_tile)
{
    tm_encode_fn encode = nullptr;
    int rc = tensor_encoder(p, &encode);
    if (rc != VL_OK) return rc;
    const cuuint64_t dims[3] = {256, nfull, n};
    const cuuint64_t strides[2] = {512, pitch * 2};
    const cuuint32_t box[3] = {256, chunks_per_tile, 8};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = encode(tm, CU_TENSOR_MAP_DATA_TYPE_UINT16, 3, (void *)d_cand, dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { p->last_cuda_error = (int)cudaErrorInvalidValue; return VL_ERR_CUDA; }
    return VL_OK;
}

// The tables of one pass as a 3-D tensor for the tiled stores of k_tables8: [groups][V + 1 vregs][64 candidates],
// a box = 8 candidates (16 bytes) x `rows` vregs of one group.
int encode_tg_tensor(vl_program *p, CUtensorMap *tm, uint16_t *tg, uint32_t groups, uint32_t rows)
{
    tm_encode_fn encode = nullptr;
    int rc = tensor_encoder(p, &encode);
    if (rc != VL_OK) return rc;
    const cuuint64_t dims[3] = {TGW, (cuuint64_t)p->V + 1, groups};
    const cuuint64_t strides[2] = {TGW * 2, ((cuuint64_t)p->V + 1) * TGW * 2};
    const cuuint32_t box[3] = {8, rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = encode(tm, CU_TENSOR_MAP_DATA_TYPE_UINT16, 3, (void *)tg, dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { p->last_cuda_error = (int)cudaErrorInvalidValue; return VL_ERR_CUDA; }
    return VL_OK;
}

template <int G, int NT>
cudaError_t launch_tables(const TParams &q, uint32_t grid, uint32_t smem, cudaStream_t st)
{
    k_tables<G, NT><<<grid, NT, smem, st>>>(q);
    return cudaGetLastError();
}

// Most work items one candidate can list for the recount: every chunk in RC_PARTS pieces, the bank
// tally in RC_BANK_PARTS slices, one item per block whose through-set collided (through-sets are
// used only by programs of at most 32 blocks).
uint64_t rc_items_per_row(const vl_program *p)
{
    return (uint64_t)RC_PARTS * p->nC + RC_BANK_PARTS + std::min<uint32_t>(p->nB, 32u);
}

int ensure_scratch(vl_program *p, int slot, uint64_t rows)
{
    vl_program::VScratch &v = p->vs[slot];
    const uint64_t aw = std::max(1u, (p->nC + 31) / 32);
    const uint64_t groups = (rows + TGW - 1) / TGW;
    if (v.rows >= rows && v.aw == aw && v.vregs == p->V && v.chunks == p->nC) return VL_OK;
    cudaFree(v.tg); cudaFree(v.cstate); cudaFree(v.anom); cudaFree(v.work); cudaFree(v.racc); cudaFree(v.grp_done); cudaFree(v.thm);
    v.tg = nullptr; v.cstate = nullptr; v.anom = nullptr; v.work = nullptr; v.racc = nullptr; v.grp_done = nullptr; v.thm = nullptr;
    v.rows = 0;
    VL_CUDA(p, cudaMalloc((void **)&v.tg, groups * (p->V + 1) * TGW * sizeof(uint16_t)));
    VL_CUDA(p, cudaMemset(v.tg, 0, groups * (p->V + 1) * TGW * sizeof(uint16_t)));
    VL_CUDA(p, cudaMalloc((void **)&v.cstate, groups * TGW * 8 * sizeof(uint32_t)));
    VL_CUDA(p, cudaMemset(v.cstate, 0, groups * TGW * 8 * sizeof(uint32_t)));
    VL_CUDA(p, cudaMalloc((void **)&v.anom, groups * TGW * aw * sizeof(uint32_t)));
    VL_CUDA(p, cudaMalloc((void **)&v.work, (RC_HDR + 2 * groups * TGW * rc_items_per_row(p)) * sizeof(uint32_t)));
    VL_CUDA(p, cudaMalloc((void **)&v.racc, groups * TGW * 4 * sizeof(uint32_t)));
    // walk blocks finished per group, then the groups' straddle-mark flags (reset by the walk)
    VL_CUDA(p, cudaMalloc((void **)&v.grp_done, 2 * (groups + 1) * sizeof(uint32_t)));
    VL_CUDA(p, cudaMemset(v.grp_done, 0, 2 * (groups + 1) * sizeof(uint32_t)));
    // through-set masks of every (group, program block), in the walk's layout
    VL_CUDA(p, cudaMalloc((void **)&v.thm, std::max<uint64_t>(1, groups * p->nB * ((p->P + p->wmax + 31) / 32) * 64) * sizeof(uint32_t)));
    v.rows = groups * TGW;
    v.aw = aw;
    v.vregs = p->V;
    v.chunks = p->nC;
    return VL_OK;
}
}  // namespace

// Records the next timing event of the handle on `st` (no-op unless kernel timing is switched on).
static void kt_mark(vl_program *p, cudaStream_t st)
{
    if (!p->ktime || p->kt_used >= 5 * 4096) return;
    if (p->kt_used == p->kt_ev.size()) {
        cudaEvent_t ev;
        if (cudaEventCreate(&ev) != cudaSuccess) { p->ktime = 0; return; }
        p->kt_ev.push_back(ev);
    }
    cudaEventRecord(p->kt_ev[p->kt_used++], st);
}

namespace {
struct PassPlan {
    Plan pl;
    uint32_t Wp, ev_cap, walk_smem, walk_warps, rc_smem;
    uint64_t sub;
};

// Launch geometry of a program's passes and the shared-memory opt-ins of its kernels.
int plan_passes(vl_program *p, uint64_t K, PassPlan *pp)
{
    const uint32_t SM_BYTES = 227 * 1024;
    // preference: eight candidates per block (two blocks of 256 threads per SM if the tables are small,
    // else one block of 512 threads), then the largest group that still lets two blocks share an SM,
    // then anything that fits
    Plan pl{};
    const uint32_t groups[3] = {4, 2, 1};
    const uint32_t NT = p->threads_opt ? p->threads_opt : 256;
    if (p->group_opt == 0 || p->group_opt == 8) {
        pl = make_plan8(p, p->threads_opt ? p->threads_opt : 256, SM_BYTES / 2 - 1024);
        if (!pl.ok) pl = make_plan8(p, p->threads_opt ? p->threads_opt : 512, SM_BYTES);
        if (!pl.ok && !p->threads_opt) pl = make_plan8(p, 256, SM_BYTES);
    }
    for (int pass = 0; pass < 2 && !pl.ok; ++pass)
        for (uint32_t G : groups) {
            if (p->group_opt && G != p->group_opt) continue;
            pl = make_plan(p, G, NT, pass == 0 ? (SM_BYTES / 2 - 1024) : SM_BYTES);
            if (pl.ok) break;
        }
    if (!pl.ok) return VL_ERR_UNSUPPORTED;
    pp->pl = pl;
    pp->Wp = (p->P + p->wmax + 31) / 32;
    pp->ev_cap = 256;
    // the walk's warps each keep the occupancy masks of 64 candidates: fewer warps for large register files
    for (pp->walk_warps = WALK_WARPS;; pp->walk_warps >>= 1) {
        pp->walk_smem = pp->walk_warps * (pp->Wp * 64 + ((pp->ev_cap >> 3) + 2) * 28) * 4;
        if (pp->walk_smem <= SM_BYTES - 1024) break;
        if (pp->walk_warps == 1) return VL_ERR_UNSUPPORTED;
    }
    // the recount keeps one cache word per vreg in shared memory when that leaves room for several
    // thread blocks per SM, else it fetches from global memory every time
    pp->rc_smem = (uint64_t)p->V * 4 <= 72 * 1024
                      ? (uint32_t)align16(((uint64_t)(p->V + 4) + 2ull * (p->P + p->wmax + 2)) * 4) : 0u;
    // the walk's table entries keep bit 15 for a mark: every in-file register number must be below 2^15
    // (the occupancy masks of a register file that large would not fit shared memory anyway)
    if (p->P + p->wmax > 32768u) return VL_ERR_UNSUPPORTED;
    // the recount work list holds up to rc_items_per_row items per candidate: keep it within 8 Mi items
    const uint64_t sub_cap = std::max<uint64_t>(32, ((8ull << 20) / rc_items_per_row(p)) / 32 * 32);
    pp->sub = std::min<uint64_t>(K, std::min<uint64_t>(p->sub_batch, sub_cap));
    // passes of equal size (whole groups of the tables) rather than full ones and a short last one
    if (K > pp->sub) {
        const uint64_t n_pass = (K + pp->sub - 1) / pp->sub;
        const uint64_t even = ((K + n_pass - 1) / n_pass + TGW - 1) / TGW * TGW;
        pp->sub = std::min(pp->sub, even);
    }
    // once per device: every verify kernel may use the whole shared memory of an SM
    static std::mutex attr_mutex;
    static bool attr_done[64];
    if (p->device >= 0 && p->device < 64) {
        std::lock_guard<std::mutex> lock(attr_mutex);
        if (!attr_done[p->device]) {
            const int sm = (int)SM_BYTES;
            const cudaFuncAttribute at = cudaFuncAttributeMaxDynamicSharedMemorySize;
            // (the walk and the recount also have a few bytes of static shared memory)
            cudaError_t e = cudaFuncSetAttribute(k_walk, at, sm - 1024);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(k_through, at, sm - 1024);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(k_recount<true>, at, sm - 1024);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tables<4, 256>, at, sm);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tables<2, 256>, at, sm);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tables<1, 256>, at, sm);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tables<4, 512>, at, sm);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tables<2, 512>, at, sm);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tables<1, 512>, at, sm);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tables8<256>, at, sm);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tables8<512>, at, sm);
            if (e != cudaSuccess) { p->last_cuda_error = (int)e; return VL_ERR_CUDA; }
            attr_done[p->device] = true;
        }
    }
    return VL_OK;
}

// One pass: the four kernels over n <= sub candidates, in order on `st`, with working set `slot`.
int run_pass(vl_program *p, const PassPlan &pp, const uint16_t *d_cand, uint64_t n, uint64_t pitch, vl_verdict *d_out,
             cudaStream_t st, int slot, bool dict, bool stagger)
{
    // what the rows hold: one column per operand occurrence, or one per dictionary entry
    const uint32_t nO = dict ? p->nD : p->nO, nOp8 = dict ? p->nD8 : p->nOp8;
    const Plan &pl = pp.pl;
    int rc = ensure_scratch(p, slot, pp.sub);
    if (rc != VL_OK) return rc;
    vl_program::VScratch &vs = p->vs[slot];
    cudaError_t e = cudaSuccess;
    const uint32_t ngrp = (uint32_t)((n + TGW - 1) / TGW);

    TParams tq{};
    tq.nI = p->nI; tq.V = p->V; tq.nO = nO; tq.nOp8 = nOp8; tq.P = p->P; tq.Bmask = p->B - 1;
    tq.ntiles = (nOp8 + pl.NT * 8 - 1) / (pl.NT * 8);
    tq.bank_fast = p->bank_fast;
    tq.vreg16 = dict ? p->d_dict_vreg16 : p->d_vreg16; tq.slotmeta = dict ? p->d_dict_slotmeta : p->d_slotmeta;
    tq.vinfo = p->d_vinfo;
    tq.entry_instr = dict ? p->d_dict_instr : nullptr;
    tq.first_def_instr = p->d_first_def_instr; tq.op_off = p->d_op_off;
    tq.bank_list = p->d_bank_list;
    for (int j = 0; j < 4; ++j) tq.bank_seg[j] = p->bank_seg[j];
    tq.bank_total = 2 * (p->bank_seg[1] - p->bank_seg[0]) + 3 * (p->bank_seg[2] - p->bank_seg[1]) +
                    4 * (p->bank_seg[3] - p->bank_seg[2]);
    tq.cand = d_cand; tq.K = n; tq.pitch = pitch;
    tq.tg = vs.tg; tq.cstate = vs.cstate; tq.status = p->d_status + 1;
    tq.NS = pl.NS; tq.off_region = pl.off_region; tq.off_misc = pl.off_misc;
    tq.AW = (uint32_t)vs.aw; tq.anom = vs.anom; tq.racc = vs.racc; tq.grp_done = vs.grp_done; tq.work = vs.work;
    tq.vcons = p->d_vcons; tq.rs_prefix = p->d_rs_prefix;
    tq.opoff = dict ? p->d_dict_opoff : p->d_opoff; tq.first4 = dict ? p->d_dict_first4 : p->d_first4;
    tq.grp_flag = vs.grp_done + (vs.rows / TGW + 1);
    tq.test_wait = p->test_wait;
    tq.pf = p->prefetch_tiles;
    tq.stagger_ns = stagger ? p->stagger_us * 1000u : 0u;
    tq.stagger_blocks = (uint32_t)vl_sm_count(p);
    const uint32_t tgrid = (uint32_t)((n + pl.G - 1) / pl.G);
    kt_mark(p, st);
    if (pl.G == 8) {
        tq.ntiles = (nOp8 + pl.NT * 4 - 1) / (pl.NT * 4);
        tq.nfull = nOp8 / 256;
        tq.tail_start = tq.nfull * 256;
        tq.tail_tile = tq.tail_start / (pl.NT * 4);
        tq.off_tail = pl.off_tail;
        alignas(64) CUtensorMap tm;
        memset(&tm, 0, sizeof(tm));
        if (tq.nfull) {
            rc = encode_row_tensor(p, &tm, d_cand, n, pitch, tq.nfull, pl.NT * 4 / 256);
            if (rc != VL_OK) return rc;
        }
        alignas(64) CUtensorMap tmg;
        tq.tg_rows = std::min<uint32_t>(256u, p->V + 1);
        rc = encode_tg_tensor(p, &tmg, vs.tg, ngrp, tq.tg_rows);
        if (rc != VL_OK) return rc;
        if (pl.NT == 256) k_tables8<256><<<tgrid, 256 + 32, pl.smem, st>>>(tq, tm, tmg);
        else k_tables8<512><<<tgrid, 512 + 32, pl.smem, st>>>(tq, tm, tmg);
        e = cudaGetLastError();
    } else if (pl.NT == 256) {
        if (pl.G == 4) e = launch_tables<4, 256>(tq, tgrid, pl.smem, st);
        else if (pl.G == 2) e = launch_tables<2, 256>(tq, tgrid, pl.smem, st);
        else e = launch_tables<1, 256>(tq, tgrid, pl.smem, st);
    } else {
        if (pl.G == 4) e = launch_tables<4, 512>(tq, tgrid, pl.smem, st);
        else if (pl.G == 2) e = launch_tables<2, 512>(tq, tgrid, pl.smem, st);
        else e = launch_tables<1, 512>(tq, tgrid, pl.smem, st);
    }
    if (e != cudaSuccess) { p->last_cuda_error = (int)e; return VL_ERR_CUDA; }
    g_vl_launches.fetch_add(1);

    kt_mark(p, st);
    // Everything from here on reads what vl_liveness computes (through-sets, walk events, live-after
    // lists); the table kernel above reads the program's operand tables only and may run beside a
    // liveness run that is still in flight.
    if ((rc = vl_live_join(p, st)) != VL_OK) return rc;
    if (p->nC) {
        WParams wq{};
        wq.V = p->V; wq.P = p->P; wq.nB = p->nB; wq.nC = p->nC; wq.Wp = pp.Wp; wq.AW = (uint32_t)vs.aw;
        wq.use_th = (uint32_t)p->use_th; wq.K = n;
        wq.th_off = p->d_th_off; wq.th = p->d_th; wq.cev_off = p->d_cev_off; wq.ev = p->d_ev;
        // the through-set masks come from a kernel of their own, except for small jobs
        const bool own_through = p->use_th && n >= 512;
        wq.thm = own_through ? vs.thm : nullptr;
        wq.tg = vs.tg; wq.ev_cap = pp.ev_cap; wq.wmax = p->wmax;
        wq.cstate = vs.cstate; wq.anom = vs.anom;
        wq.grp_flag = vs.grp_done + (vs.rows / TGW + 1);
        wq.list_all = p->bank_fast ? 0 : 1; wq.chunk_blk = p->d_chunk_blk;
        wq.grp_done = vs.grp_done; wq.work = vs.work; wq.racc = vs.racc; wq.out = d_out;
        if (own_through) {
            k_through<<<dim3(p->nB, ngrp), 256, pp.Wp * 64 * 4, st>>>(wq);
            e = cudaGetLastError();
            if (e != cudaSuccess) { p->last_cuda_error = (int)e; return VL_ERR_CUDA; }
            g_vl_launches.fetch_add(1);
        }
        const dim3 wgrid((p->nC + pp.walk_warps - 1) / pp.walk_warps, ngrp);
        k_walk<<<wgrid, pp.walk_warps * 32, pp.walk_smem, st>>>(wq);
        e = cudaGetLastError();
        if (e != cudaSuccess) { p->last_cuda_error = (int)e; return VL_ERR_CUDA; }
        g_vl_launches.fetch_add(1);
    }

    // programs whose bank tally cannot take the fast path (banks not 1, 2 or 4, or an instruction
    // with more than 4 distinct sources) send every candidate through k_recount
    kt_mark(p, st);
    if (!p->nC) {  // nothing to walk: the verdict step runs on its own
        k_finish<<<(uint32_t)((n * 32 + 127) / 128), 128, 0, st>>>(n, p->nC, (uint32_t)vs.aw, p->bank_fast ? 0 : 1,
                                                                  vs.cstate, vs.anom, p->d_chunk_blk, vs.work, vs.racc,
                                                                  d_out);
        g_vl_launches.fetch_add(1);
    }
    RParams rq{};
    rq.nI = p->nI; rq.V = p->V; rq.B = p->B; rq.nB = p->nB; rq.nC = p->nC; rq.AW = (uint32_t)vs.aw;
    rq.bank_fast = p->bank_fast; rq.K = n;
    rq.blk_chunk_off = p->d_blk_chunk_off; rq.th_off = p->d_th_off; rq.th = p->d_th;
    rq.el = p->d_el; rq.el_count = p->d_el_count;
    rq.ls = p->d_ls; rq.ls_adj = p->d_ls_adj; rq.th_cnt = p->d_th_cnt; rq.R = p->P + p->wmax + 2;
    rq.vinfo = p->d_vinfo; rq.chunk_i0 = p->d_chunk_i0; rq.chunk_i1 = p->d_chunk_i1; rq.chunk_blk = p->d_chunk_blk;
    rq.op_off = p->d_op_off; rq.op_vreg = p->d_op_vreg; rq.lo_off = p->d_lo_off; rq.lo = p->d_lo;
    rq.ndefs = p->d_ndefs; rq.width = p->d_width; rq.opflags = p->d_opflags; rq.iflags = p->d_iflags;
    rq.racc = vs.racc; rq.status = p->d_status + 1;
    rq.tg = vs.tg; rq.cstate = vs.cstate; rq.anom = vs.anom; rq.work = vs.work; rq.out = d_out;
    rq.bank_list = p->d_bank_list;
    for (int j = 0; j < 4; ++j) rq.bank_seg[j] = p->bank_seg[j];
    const uint32_t rgrid = (uint32_t)vl_sm_count(p) * 6;  // thread blocks of the recount: they take items from a shared cursor
    kt_mark(p, st);
    if (pp.rc_smem) k_recount<true><<<rgrid, RC_THREADS, pp.rc_smem, st>>>(rq);
    else k_recount<false><<<rgrid, RC_THREADS, 0, st>>>(rq);
    kt_mark(p, st);
    e = cudaGetLastError();
    if (e != cudaSuccess) { p->last_cuda_error = (int)e; return VL_ERR_CUDA; }
    g_vl_launches.fetch_add(1);
    return VL_OK;
}
}  // namespace

// All passes in order on one stream, with one working set.
int vl_verify_impl(vl_program *p, const uint16_t *d_cand, uint64_t K, uint64_t pitch, vl_verdict *d_out,
                   cudaStream_t st, int slot, bool dict)
{
    PassPlan pp{};
    int rc = plan_passes(p, K, &pp);
    if (rc != VL_OK) return rc;
    for (uint64_t kb = 0; kb < K; kb += pp.sub) {
        rc = run_pass(p, pp, d_cand + kb * pitch, std::min(pp.sub, K - kb), pitch, d_out + kb, st, slot, dict,
                      kb == 0 && K >= 8ull * 2 * (uint64_t)vl_sm_count(p));
        if (rc != VL_OK) return rc;
    }
    return VL_OK;
}

// Passes of one or several programs spread round-robin over the device's lane streams, so that
// the table kernel of one pass (bound by the row stream) runs beside the walk of another (bound by
// instruction issue).  Pass j of a program uses working set j mod lanes and runs on lane
// (first_lane + j) mod lanes: two passes that share a working set are ordered by their stream.
int vl_verify_lanes(uint32_t nprog, vl_program *const *progs, const uint16_t *const *d_cand, const uint64_t *K,
                    const uint64_t *pitch, vl_verdict *const *d_out, cudaStream_t st, bool dict)
{
    vl_program *p0 = progs[0];
    cudaStream_t *lane = nullptr;
    int rc = vl_lane_streams(p0, &lane);
    if (rc != VL_OK) return rc;
    // several programs in one call are small jobs bound by launch latency: they take every lane
    const uint32_t L = p0->lanes_opt == 1 ? 1u : (nprog > 1 ? (uint32_t)VL_LANES : std::min<uint32_t>(VL_LANES, p0->lanes_opt));
    uint64_t jobs = 0;
    for (uint32_t j = 0; j < nprog; ++j) jobs += (K[j] + progs[j]->sub_batch - 1) / progs[j]->sub_batch;
    if (L == 1 || jobs <= 1) {
        for (uint32_t j = 0; j < nprog; ++j) {
            if (K[j] == 0) continue;
            rc = vl_verify_impl(progs[j], d_cand[j], K[j], pitch[j], d_out[j], st, 0, dict);
            if (rc != VL_OK) return rc;
        }
        return VL_OK;
    }
    VL_CUDA(p0, cudaEventRecord(p0->ev_fork, st));
    for (uint32_t l = 0; l < L; ++l) VL_CUDA(p0, cudaStreamWaitEvent(lane[l], p0->ev_fork, 0));
    uint64_t job = 0;
    for (uint32_t j = 0; j < nprog && rc == VL_OK; ++j) {
        if (K[j] == 0) continue;
        vl_program *p = progs[j];
        PassPlan pp{};
        rc = plan_passes(p, K[j], &pp);
        if (rc != VL_OK) break;
        // a program's passes keep to "working set s on lane (base + s) mod L"
        const uint64_t base = job;
        uint64_t s = 0;
        for (uint64_t kb = 0; kb < K[j] && rc == VL_OK; kb += pp.sub, ++s, ++job)
            rc = run_pass(p, pp, d_cand[j] + kb * pitch[j], std::min(pp.sub, K[j] - kb), pitch[j], d_out[j] + kb,
                          lane[(base + s) % L], (int)(s % L), dict, job == 0 && K[j] >= 8ull * 2 * (uint64_t)vl_sm_count(p));
    }
    // join even after an error, so that the caller's stream stays ordered after what was launched
    for (uint32_t l = 0; l < L; ++l) {
        cudaError_t e = cudaEventRecord(p0->ev_join[l], lane[l]);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, p0->ev_join[l], 0);
        if (e != cudaSuccess && rc == VL_OK) { p0->last_cuda_error = (int)e; rc = VL_ERR_CUDA; }
    }
    return rc;
}
