// Liveness on the GPU and the per-program tables the verify kernels consume.
//
// Pipeline (all kernels on the caller's stream).  Every block is cut into chunks (the unit of the
// verify walk) and every chunk into pieces of at most PIECE_INSTRS instructions (the unit of the
// backward instruction walk here, so that a few thousand warps share it):
//   piece read/write sets -> chunk sets -> block sets -> fixed point over blocks (one thread per
//   bitset word) -> live set at every chunk boundary -> at every piece boundary -> backward walk
//   of every piece (count, then fill) giving the per-instruction live-after lists in CSR form and
//   the per-operand flags -> operand metadata, walk events, through-sets.
#include <algorithm>
#include <cstring>
#include <vector>

#include "vl_internal.cuh"

#define NT 128  // threads per block in every kernel of this file
#define PIECE_INSTRS 8
#ifndef VL_ITEM_CHUNKS
#define VL_ITEM_CHUNKS 32  // chunks per walk work item
#endif

// ------------------------------------------------------------------ device helpers
__device__ __forceinline__ bool bit_get(const uint32_t *s, uint32_t v) { return (s[v >> 5] >> (v & 31)) & 1u; }
__device__ __forceinline__ void bit_set(uint32_t *s, uint32_t v) { s[v >> 5] |= 1u << (v & 31); }
__device__ __forceinline__ void bit_clr(uint32_t *s, uint32_t v) { s[v >> 5] &= ~(1u << (v & 31)); }

// Exclusive scan over the NT threads of a block; *total gets the block sum.
// s_scan needs 34 words.  Contains barriers: every thread of the block must call it.
__device__ uint32_t block_excl_scan(uint32_t x, uint32_t *s_scan, uint32_t *total)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    uint32_t inc = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t y = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += y;
    }
    __syncthreads();  // protects s_scan against readers of a previous call
    if (lane == 31) s_scan[w] = inc;
    __syncthreads();
    if (w == 0) {
        uint32_t t = lane < NT / 32 ? s_scan[lane] : 0u;
        uint32_t ti = t;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            uint32_t y = __shfl_up_sync(0xffffffffu, ti, d);
            if (lane >= d) ti += y;
        }
        if (lane < NT / 32) s_scan[lane] = ti - t;
        if (lane == 31) s_scan[33] = ti;
    }
    __syncthreads();
    *total = s_scan[33];
    return s_scan[w] + inc - x;
}

// Calls emit(rank, bit index) for every set bit of words[0..nwords), ranks ascending with
// the bit index.  Contains barriers.
template <class F>
__device__ void compact_bits(const uint32_t *words, uint32_t nwords, uint32_t *s_scan, uint32_t *total, F emit)
{
    const uint32_t per = (nwords + NT - 1) / NT;
    const uint32_t w0 = min(nwords, threadIdx.x * per), w1 = min(nwords, w0 + per);
    uint32_t cnt = 0;
    for (uint32_t w = w0; w < w1; ++w) cnt += __popc(words[w]);
    uint32_t off = block_excl_scan(cnt, s_scan, total);
    for (uint32_t w = w0; w < w1; ++w) {
        uint32_t x = words[w];
        while (x) {
            uint32_t b = __ffs(x) - 1;
            x &= x - 1;
            emit(off++, w * 32 + b);
        }
    }
}

// ------------------------------------------------------------------------- kernels
// Per span of instructions (a piece): use = vregs read before any write inside the span, def = vregs written.
__global__ void k_chunk_sets(const uint32_t *__restrict__ chunk_i0, const uint32_t *__restrict__ chunk_i1,
                             const uint32_t *__restrict__ op_off, const uint8_t *__restrict__ ndefs,
                             const uint32_t *__restrict__ op_vreg, uint32_t Wv, uint32_t *chunk_use,
                             uint32_t *chunk_def)
{
    extern __shared__ uint32_t sm[];
    uint32_t *s_use = sm, *s_def = sm + Wv;
    const uint32_t c = blockIdx.x;
    for (uint32_t w = threadIdx.x; w < 2 * Wv; w += NT) sm[w] = 0;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (uint32_t i = chunk_i0[c]; i < chunk_i1[c]; ++i) {
            const uint32_t o0 = op_off[i], o1 = op_off[i + 1], nd = ndefs[i];
            for (uint32_t o = o0 + nd; o < o1; ++o) {  // reads first
                uint32_t v = op_vreg[o];
                if (!bit_get(s_def, v)) bit_set(s_use, v);
            }
            for (uint32_t o = o0; o < o0 + nd; ++o) bit_set(s_def, op_vreg[o]);
        }
    }
    __syncthreads();
    for (uint32_t w = threadIdx.x; w < Wv; w += NT) {
        chunk_use[(size_t)c * Wv + w] = s_use[w];
        chunk_def[(size_t)c * Wv + w] = s_def[w];
    }
}

// Per parent (a block over its chunks, a chunk over its pieces): compose the children's sets in order.
__global__ void k_block_sets(const uint32_t *__restrict__ blk_chunk_off, uint32_t Wv,
                             const uint32_t *__restrict__ chunk_use, const uint32_t *__restrict__ chunk_def,
                             uint32_t *blk_use, uint32_t *blk_def)
{
    const uint32_t b = blockIdx.y, w = blockIdx.x * NT + threadIdx.x;  // one bitset word per thread
    if (w >= Wv) return;
    const uint32_t c_lo = blk_chunk_off[b], c_hi = blk_chunk_off[b + 1];
    uint32_t u = 0, d = 0;
#pragma unroll 8
    for (uint32_t c = c_lo; c < c_hi; ++c) {
        u |= chunk_use[(size_t)c * Wv + w] & ~d;
        d |= chunk_def[(size_t)c * Wv + w];
    }
    blk_use[(size_t)b * Wv + w] = u;
    blk_def[(size_t)b * Wv + w] = d;
}

// Backward dataflow to the least fixed point.  Bitset words are independent of each other,
// so one thread iterates one word column over all blocks until nothing changes; no barrier.
// SMEM: the four sets of this thread's word column and the successor lists sit in shared memory
// ([4][nB][NT] words, then succ_off[nB + 1] and succ[nE]); otherwise everything stays in global memory.
template <bool SMEM>
__global__ void k_fixed_point(uint32_t nB, uint32_t nE, uint32_t Wv, const uint32_t *__restrict__ succ_off,
                              const uint32_t *__restrict__ succ, const uint32_t *__restrict__ blk_use,
                              const uint32_t *__restrict__ blk_def, uint32_t *live_in, uint32_t *live_out,
                              uint32_t *status)
{
    const uint32_t w = blockIdx.x * NT + threadIdx.x;
    if (SMEM) {
        extern __shared__ uint32_t fsm[];
        uint32_t *s_use = fsm, *s_def = fsm + nB * NT, *s_in = fsm + 2 * nB * NT, *s_out = fsm + 3 * nB * NT;
        uint32_t *s_so = fsm + 4 * nB * NT, *s_su = s_so + nB + 1;
        for (uint32_t i = threadIdx.x; i <= nB; i += NT) s_so[i] = succ_off[i];
        for (uint32_t i = threadIdx.x; i < nE; i += NT) s_su[i] = succ[i];
        const uint32_t t = threadIdx.x;
        for (uint32_t b = 0; b < nB; ++b) {
            s_use[b * NT + t] = w < Wv ? blk_use[(size_t)b * Wv + w] : 0u;
            s_def[b * NT + t] = w < Wv ? blk_def[(size_t)b * Wv + w] : 0u;
            s_in[b * NT + t] = 0;
            s_out[b * NT + t] = 0;
        }
        __syncthreads();
        if (w >= Wv) return;
        bool changed = true;
        for (uint32_t sweep = 0; sweep < nB + 2 && changed; ++sweep) {
            changed = false;
            for (uint32_t n = 0; n < nB; ++n) {
                const uint32_t b = nB - 1 - n;
                uint32_t o = 0;
                for (uint32_t e = s_so[b]; e < s_so[b + 1]; ++e) o |= s_in[s_su[e] * NT + t];
                const uint32_t in = s_use[b * NT + t] | (o & ~s_def[b * NT + t]);
                if (o != s_out[b * NT + t] || in != s_in[b * NT + t]) changed = true;
                s_out[b * NT + t] = o;
                s_in[b * NT + t] = in;
            }
        }
        for (uint32_t b = 0; b < nB; ++b) {
            live_in[(size_t)b * Wv + w] = s_in[b * NT + t];
            live_out[(size_t)b * Wv + w] = s_out[b * NT + t];
        }
        if (changed) atomicOr(status, ST_NO_CONVERGE);
        if (s_in[t] != 0) atomicOr(status, ST_NOT_STRICT);  // block 0 is the entry
        return;
    }
    if (w >= Wv) return;
    bool changed = true;
    for (uint32_t sweep = 0; sweep < nB + 2 && changed; ++sweep) {
        changed = false;
        for (uint32_t n = 0; n < nB; ++n) {
            const uint32_t b = nB - 1 - n;
            uint32_t o = 0;
            for (uint32_t e = succ_off[b]; e < succ_off[b + 1]; ++e) o |= live_in[(size_t)succ[e] * Wv + w];
            const uint32_t in = blk_use[(size_t)b * Wv + w] | (o & ~blk_def[(size_t)b * Wv + w]);
            if (o != live_out[(size_t)b * Wv + w] || in != live_in[(size_t)b * Wv + w]) changed = true;
            live_out[(size_t)b * Wv + w] = o;
            live_in[(size_t)b * Wv + w] = in;
        }
    }
    if (changed) atomicOr(status, ST_NO_CONVERGE);
    if (live_in[w] != 0) atomicOr(status, ST_NOT_STRICT);  // block 0 is the entry
}

// Live set after the last instruction of every child (chunk_end) and before its first (chunk_entry,
// may be null), walking a parent's children backwards from the parent's live-out set: chunks of a
// block, or pieces of a chunk.
__global__ void k_chunk_boundaries(const uint32_t *__restrict__ blk_chunk_off, uint32_t Wv,
                                   const uint32_t *__restrict__ live_out, const uint32_t *__restrict__ chunk_use,
                                   const uint32_t *__restrict__ chunk_def, uint32_t *chunk_end, uint32_t *chunk_entry)
{
    const uint32_t b = blockIdx.y, w = blockIdx.x * NT + threadIdx.x;  // one bitset word per thread
    if (w >= Wv) return;
    const uint32_t c_lo = blk_chunk_off[b], c_hi = blk_chunk_off[b + 1];
    uint32_t live = live_out[(size_t)b * Wv + w];
    if (chunk_entry) {
#pragma unroll 8
        for (uint32_t c = c_hi; c-- > c_lo;) {
            chunk_end[(size_t)c * Wv + w] = live;
            live = chunk_use[(size_t)c * Wv + w] | (live & ~chunk_def[(size_t)c * Wv + w]);
            chunk_entry[(size_t)c * Wv + w] = live;
        }
    } else {
#pragma unroll 8
        for (uint32_t c = c_hi; c-- > c_lo;) {
            chunk_end[(size_t)c * Wv + w] = live;
            live = chunk_use[(size_t)c * Wv + w] | (live & ~chunk_def[(size_t)c * Wv + w]);
        }
    }
}

// Backward walk of one piece by one warp.  FILL = false: list sizes, per-operand flags, walk-event
// counts, and the set of vregs whose occupancy changes inside the chunk.  FILL = true: the lists.
// The chunk's slice of the operand arrays is staged in shared memory when it fits (WALK_CAP_I
// instructions, WALK_CAP_O operands); lane 0 does the per-instruction bookkeeping, all lanes the
// population count / compaction of the live bitset.
#define WALK_CAP_I 32
#define WALK_CAP_O 256
template <bool FILL>
__global__ void __launch_bounds__(32) k_instr_walk(const uint32_t *__restrict__ chunk_i0,
                                                   const uint32_t *__restrict__ chunk_i1,
                                                   const uint32_t *__restrict__ op_off, const uint8_t *__restrict__ ndefs,
                                                   const uint32_t *__restrict__ op_vreg, uint32_t Wv,
                                                   const uint32_t *__restrict__ chunk_end, uint32_t *lo_cnt,
                                                   uint32_t *ev_cnt, uint8_t *opflags,
                                                   const uint32_t *__restrict__ piece_chunk, uint32_t *chunk_touch,
                                                   const uint32_t *__restrict__ lo_off, uint32_t *lo,
                                                   const uint32_t *__restrict__ chunk_blk,
                                                   const uint32_t *__restrict__ blk_th,
                                                   const uint32_t *__restrict__ ls_adj,
                                                   const uint32_t *__restrict__ th_cnt, uint32_t *ls)
{
    extern __shared__ uint32_t sm[];
    uint32_t *s_live = sm, *s_touch = sm + Wv;
    uint32_t *s_off = sm + 2 * Wv;                 // [WALK_CAP_I + 1]
    uint32_t *s_lo = s_off + WALK_CAP_I + 1;       // [WALK_CAP_I] list offsets (FILL)
    uint32_t *s_ops = s_lo + WALK_CAP_I;           // [WALK_CAP_O]
    uint8_t *s_nd = reinterpret_cast<uint8_t *>(s_ops + WALK_CAP_O);  // [WALK_CAP_I]
    const uint32_t c = blockIdx.x, lane = threadIdx.x;
    const uint32_t i0 = chunk_i0[c], i1 = chunk_i1[c];
    // FILL: second list per instruction without the vregs that stay occupied through the whole block
    // (s_touch then holds the block's through-set); every instruction of the block has all of them in
    // its live-after set, so the short list of instruction i starts at lo_off[i] - ls_adj[b] - i * th_cnt[b]
    uint32_t ls_sub = 0, ls_mul = 0;
    if (FILL) {
        const uint32_t b = chunk_blk[piece_chunk[c]];
        ls_sub = ls_adj[b];
        ls_mul = th_cnt[b];
        for (uint32_t w = lane; w < Wv; w += 32) s_touch[w] = blk_th[(size_t)b * Wv + w];
    }
    for (uint32_t w = lane; w < Wv; w += 32) {
        s_live[w] = chunk_end[(size_t)c * Wv + w];
        if (!FILL) s_touch[w] = 0;
    }
    const uint32_t ob = i1 > i0 ? op_off[i0] : 0, oe = i1 > i0 ? op_off[i1] : 0;
    const bool staged = (i1 - i0) <= WALK_CAP_I && (oe - ob) <= WALK_CAP_O;
    if (staged) {
        for (uint32_t i = i0 + lane; i <= i1; i += 32) s_off[i - i0] = op_off[i];
        for (uint32_t i = i0 + lane; i < i1; i += 32) {
            s_nd[i - i0] = ndefs[i];
            if (FILL) s_lo[i - i0] = lo_off[i];
        }
        for (uint32_t o = ob + lane; o < oe; o += 32) s_ops[o - ob] = op_vreg[o];
    }
    __syncwarp();
    auto OFF = [&](uint32_t i) { return staged ? s_off[i - i0] : op_off[i]; };
    auto ND = [&](uint32_t i) -> uint32_t { return staged ? s_nd[i - i0] : ndefs[i]; };
    auto OP = [&](uint32_t o) { return staged ? s_ops[o - ob] : op_vreg[o]; };
    const uint32_t rounds = (Wv + 31) / 32;
    for (uint32_t i = i1; i-- > i0;) {
        uint32_t total = 0;
        if (FILL) {
            // ascending ids, 32 words per round; every non-empty word is broadcast and each lane whose
            // bit is set writes its id at the rank of that bit: up to 32 consecutive stores per word
            uint32_t at = staged ? s_lo[i - i0] : lo_off[i];
            uint32_t at_s = at - ls_sub - i * ls_mul;
            for (uint32_t r = 0; r < rounds; ++r) {
                const uint32_t w = r * 32 + lane;
                const uint32_t mine = w < Wv ? s_live[w] : 0u;
                const uint32_t mine_th = w < Wv ? s_touch[w] : 0u;
                uint32_t nz = __ballot_sync(0xffffffffu, mine != 0);
                while (nz) {
                    const uint32_t src = __ffs(nz) - 1;
                    nz &= nz - 1;
                    const uint32_t x = __shfl_sync(0xffffffffu, mine, src);
                    const uint32_t y = x & ~__shfl_sync(0xffffffffu, mine_th, src);
                    const uint32_t id = (r * 32 + src) * 32 + lane, below = (1u << lane) - 1u;
                    if ((x >> lane) & 1u) lo[at + __popc(x & below)] = id;
                    if ((y >> lane) & 1u) ls[at_s + __popc(y & below)] = id;
                    at += __popc(x);
                    at_s += __popc(y);
                }
            }
        } else {
            uint32_t cnt = 0;
            for (uint32_t w = lane; w < Wv; w += 32) cnt += __popc(s_live[w]);
#pragma unroll
            for (int d = 16; d; d >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, d);
            total = cnt;
        }
        __syncwarp();
        if (lane == 0) {
            const uint32_t o0 = OFF(i), o1 = OFF(i + 1), nd = ND(i);
            if (!FILL) {
                lo_cnt[i] = total;
                uint32_t evs = 0;
                for (uint32_t o = o0 + nd; o < o1; ++o) {
                    const uint32_t v = OP(o);
                    bool dup = false;
                    for (uint32_t q = o0 + nd; q < o; ++q) dup |= (OP(q) == v);
                    const bool lv = bit_get(s_live, v);
                    const bool kill = !dup && !lv;  // a read of a vreg that stays live releases nothing
                    opflags[o] = (uint8_t)((kill ? OPF_KILL : 0) | (dup ? OPF_DUP : 0));
                    if (kill) { ++evs; bit_set(s_touch, v); }
                }
                for (uint32_t o = o0; o < o0 + nd; ++o) {
                    const uint32_t v = OP(o);
                    bool selfuse = false;
                    for (uint32_t q = o0 + nd; q < o1; ++q) selfuse |= (OP(q) == v);
                    const bool lv = bit_get(s_live, v);
                    const bool elide = selfuse && lv;
                    const bool set = lv || nd > 1;
                    const bool post = !lv && nd > 1;
                    opflags[o] = (uint8_t)(OPF_DEF | (elide ? OPF_ELIDE : 0) | (set ? OPF_SET : 0) |
                                           (post ? OPF_POST : 0) | (lv ? 0 : OPF_DEAD));
                    if (!elide) { evs += 1 + (post ? 1 : 0); bit_set(s_touch, v); }
                }
                ev_cnt[i] = evs;
            }
            for (uint32_t o = o0; o < o0 + nd; ++o) bit_clr(s_live, OP(o));
            for (uint32_t o = o0 + nd; o < o1; ++o) bit_set(s_live, OP(o));
        }
        __syncwarp();
    }
    if (!FILL) {  // the vregs whose occupancy changes somewhere in the chunk this piece belongs to
        const size_t row = (size_t)piece_chunk[c] * Wv;
        for (uint32_t w = lane; w < Wv; w += 32)
            if (s_touch[w]) atomicOr(&chunk_touch[row + w], s_touch[w]);
    }
}

// Exclusive scan of a u32 array (16-byte aligned) by one block of 1024 threads, 32 items per thread and round;
// out[n] = total (saturated), total64 exact.
// Block b of the grid scans in_b into out_b (two arrays per launch).
__global__ void __launch_bounds__(1024) k_scan(const uint32_t *__restrict__ in0, uint32_t *out0,
                                               const uint32_t *__restrict__ in1, uint32_t *out1, uint32_t n,
                                               unsigned long long *totals, uint32_t *status)
{
    const uint32_t *__restrict__ in = blockIdx.x ? in1 : in0;
    uint32_t *out = blockIdx.x ? out1 : out0;
    unsigned long long *total64 = totals + blockIdx.x;
    __shared__ uint32_t s_w[33];
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned long long carry = 0;
    constexpr int IT = 32;
    for (uint32_t base = 0; base < n; base += 1024 * IT) {
        const uint32_t i = base + tid * IT;
        uint32_t x[IT];
        if (i + IT <= n) {
#pragma unroll
            for (int j = 0; j < IT; j += 4) {
                const uint4 v = *reinterpret_cast<const uint4 *>(in + i + j);
                x[j] = v.x; x[j + 1] = v.y; x[j + 2] = v.z; x[j + 3] = v.w;
            }
        } else {
#pragma unroll
            for (int j = 0; j < IT; ++j) x[j] = i + j < n ? in[i + j] : 0u;
        }
        uint32_t mine = 0;
#pragma unroll
        for (int j = 0; j < IT; ++j) mine += x[j];
        uint32_t inc = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, inc, d);
            if (lane >= d) inc += y;
        }
        __syncthreads();
        if (lane == 31) s_w[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const uint32_t t = s_w[lane];
            uint32_t ti = t;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t y = __shfl_up_sync(0xffffffffu, ti, d);
                if (lane >= d) ti += y;
            }
            s_w[lane] = ti - t;
            if (lane == 31) s_w[32] = ti;
        }
        __syncthreads();
        uint32_t ex = (uint32_t)carry + s_w[warp] + inc - mine;
        if (i + IT <= n) {
#pragma unroll
            for (int j = 0; j < IT; j += 4) {
                uint4 v;
                v.x = ex; ex += x[j];
                v.y = ex; ex += x[j + 1];
                v.z = ex; ex += x[j + 2];
                v.w = ex; ex += x[j + 3];
                *reinterpret_cast<uint4 *>(out + i + j) = v;
            }
        } else {
#pragma unroll
            for (int j = 0; j < IT; ++j) {
                if (i + j < n) out[i + j] = ex;
                ex += x[j];
            }
        }
        carry += s_w[32];
    }
    if (tid == 0) {
        out[n] = carry > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)carry;
        *total64 = carry;
        if (carry > 0xFFFFFFF0ull) atomicOr(status, ST_SIZE_OVERFLOW);
    }
}

// Through-set of a block: live on entry and never touched by a walk event inside it.
__global__ void k_block_through(const uint32_t *__restrict__ blk_chunk_off, uint32_t Wv, int use_th,
                                const uint32_t *__restrict__ live_in, const uint32_t *__restrict__ chunk_touch,
                                uint32_t *blk_th)
{
    const uint32_t b = blockIdx.y, w = blockIdx.x * NT + threadIdx.x;  // one bitset word per thread
    if (w >= Wv) return;
    const uint32_t c_lo = blk_chunk_off[b], c_hi = blk_chunk_off[b + 1];
    uint32_t t = 0;
#pragma unroll 8
    for (uint32_t c = c_lo; c < c_hi; ++c) t |= chunk_touch[(size_t)c * Wv + w];
    blk_th[(size_t)b * Wv + w] = use_th ? (live_in[(size_t)b * Wv + w] & ~t) : 0u;
}

// chunk_entry &= ~through(block); entry count; events of the chunk = entries + instruction events.
__global__ void k_chunk_entry(const uint32_t *__restrict__ chunk_blk, const uint32_t *__restrict__ chunk_i0,
                              const uint32_t *__restrict__ chunk_i1, uint32_t Wv,
                              const uint32_t *__restrict__ blk_th, uint32_t *chunk_entry,
                              const uint32_t *__restrict__ ev_off, uint32_t *centry_cnt, uint32_t *cev)
{
    __shared__ uint32_t s_scan[34];
    const uint32_t c = blockIdx.x, b = chunk_blk[c];
    uint32_t cnt = 0;
    for (uint32_t w = threadIdx.x; w < Wv; w += NT) {
        const uint32_t x = chunk_entry[(size_t)c * Wv + w] & ~blk_th[(size_t)b * Wv + w];
        chunk_entry[(size_t)c * Wv + w] = x;
        cnt += __popc(x);
    }
    uint32_t total;
    block_excl_scan(cnt, s_scan, &total);
    if (threadIdx.x == 0) {
        centry_cnt[c] = total;
        cev[c] = total + (ev_off[chunk_i1[c]] - ev_off[chunk_i0[c]]);
    }
}

__global__ void k_row_popc(uint32_t Wv, const uint32_t *__restrict__ rows, uint32_t *cnt)
{
    __shared__ uint32_t s_scan[34];
    const uint32_t r = blockIdx.x;
    uint32_t c = 0;
    for (uint32_t w = threadIdx.x; w < Wv; w += NT) c += __popc(rows[(size_t)r * Wv + w]);
    uint32_t total;
    block_excl_scan(c, s_scan, &total);
    if (threadIdx.x == 0) cnt[r] = total;
}

// Per instruction: vreg id per operand (16 bit), first occurrence / first definition of every
// vreg, and the bank-compare distances of every read.
__global__ void k_first_occ(uint32_t nI, const uint32_t *__restrict__ op_off, const uint8_t *__restrict__ ndefs,
                            const uint32_t *__restrict__ op_vreg, uint32_t *first_occ, uint32_t *first_def_instr)
{
    const uint32_t i = blockIdx.x * NT + threadIdx.x;
    if (i >= nI) return;
    const uint32_t o0 = op_off[i], o1 = op_off[i + 1], nd = ndefs[i];
    for (uint32_t o = o0; o < o1; ++o) {
        atomicMin(&first_occ[op_vreg[o]], o);
        if (o < o0 + nd) atomicMin(&first_def_instr[op_vreg[o]], i);
    }
}

__global__ void k_vreg_info(uint32_t V, const uint8_t *__restrict__ width, const uint32_t *__restrict__ first_occ,
                            const uint32_t *__restrict__ first_def_instr, uint32_t *vinfo)
{
    const uint32_t v = blockIdx.x * NT + threadIdx.x;
    if (v >= V) return;
    vinfo[v] = width[v] | (first_occ[v] != 0xFFFFFFFFu ? VINFO_OCCURS : 0u) |
               (first_def_instr[v] != 0xFFFFFFFFu ? VINFO_DEFINED : 0u);
}

// Per instruction: 1 if it has a definition the walk skips (a vreg redefined from itself while it
// stays occupied); the recount visits only those when a block's through-set collided.
__global__ void k_instr_flags(uint32_t nI, const uint32_t *__restrict__ op_off, const uint8_t *__restrict__ ndefs,
                              const uint8_t *__restrict__ opflags, uint8_t *iflags)
{
    const uint32_t i = blockIdx.x * NT + threadIdx.x;
    if (i >= nI) return;
    uint8_t f = 0;
    for (uint32_t o = op_off[i]; o < op_off[i] + ndefs[i]; ++o)
        if (opflags[o] & OPF_ELIDE) f = 1;
    iflags[i] = f;
}

// Every event slot starts as a no-op (see put_event for the layout of a group of 8 events).
__global__ void k_fill_noop(uint4 *dst, size_t n_groups, uint32_t spare_vreg)
{
    const uint32_t vv = spare_vreg * 128u, ww = 31u | (31u << 16);
    for (size_t i = (size_t)blockIdx.x * NT + threadIdx.x; i < n_groups * 7; i += (size_t)gridDim.x * NT) {
        const uint32_t part = (uint32_t)(i % 7);
        dst[i] = part < 2 ? make_uint4(vv, vv, vv, vv) : (part == 6 ? make_uint4(ww, ww, ww, ww) : make_uint4(0, 0, 0, 0));
    }
}

__global__ void k_operand_meta(uint32_t nI, const uint32_t *__restrict__ op_off, const uint8_t *__restrict__ ndefs,
                               const uint32_t *__restrict__ op_vreg, const uint32_t *__restrict__ first_occ,
                               const uint8_t *__restrict__ opflags, uint16_t *vreg16, uint8_t *opmeta,
                               uint32_t *status)
{
    const uint32_t i = blockIdx.x * NT + threadIdx.x;
    if (i >= nI) return;
    const uint32_t o0 = op_off[i], o1 = op_off[i + 1], nd = ndefs[i];
    for (uint32_t o = o0; o < o1; ++o) {
        const uint32_t v = op_vreg[o];
        uint8_t m = (first_occ[v] == o) ? 1 : 0;
        if (o >= o0 + nd && !(opflags[o] & OPF_DUP)) {
            const uint32_t u = o - (o0 + nd);  // reads of this instruction before this one
            if (u >= 1) m |= 2;
            if (u >= 2) m |= 4;
            if (u >= 3) m |= 8;
        }
        vreg16[o] = (uint16_t)v;
        opmeta[o] = m;
    }
}

// Per 8 operands: bits 0..7 first occurrence; for d = 1..3 a 16-bit field at 8 + 16 (d-1) with
// bit 2 j set when operand j compares its bank with the operand d places before it.
// Also the operand metadata of the eight-candidate table kernel, per four operands: the byte offsets
// of the vregs' 16-byte table entries and a nibble of first-occurrence bits; there, operands beyond
// n_operands (the arrays are padded to whole tiles) name the spare entry V and are never a first
// occurrence.  One thread per 8 operands of the padded arrays.
__global__ void k_pack_slots(uint32_t nO, uint32_t nOp8, uint32_t n_slots_padded, uint32_t V,
                             const uint8_t *__restrict__ opmeta, uint16_t *vreg16, uint64_t *slotmeta, uint4 *opoff,
                             uint8_t *first4)
{
    const uint32_t s = blockIdx.x * NT + threadIdx.x;
    if (s >= n_slots_padded) return;
    uint64_t m = 0;
    uint32_t off[8], f = 0;
    for (uint32_t j = 0; j < 8; ++j) {
        const uint32_t o = s * 8 + j;
        off[j] = V * 16u;
        if (o >= nO) {
            if (o < nOp8) {
                vreg16[o] = (uint16_t)V;  // padding operand: writes the spare table entry, never compared
                m |= 1ull << j;
            }
            continue;
        }
        off[j] = (uint32_t)vreg16[o] * 16u;
        const uint8_t x = opmeta[o];
        if (x & 1) { m |= 1ull << j; f |= 1u << j; }
        if (x & 2) m |= 1ull << (8 + 2 * j);
        if (x & 4) m |= 1ull << (24 + 2 * j);
        if (x & 8) m |= 1ull << (40 + 2 * j);
    }
    if (s < nOp8 / 8) slotmeta[s] = m;
    opoff[2 * s] = make_uint4(off[0], off[1], off[2], off[3]);
    opoff[2 * s + 1] = make_uint4(off[4], off[5], off[6], off[7]);
    first4[2 * s] = (uint8_t)(f & 15u);
    first4[2 * s + 1] = (uint8_t)(f >> 4);
}

// Walk events are stored in groups of 8, 112 bytes per group, field by field so that the walk
// fetches a group with 16-byte loads: off[8] (32 bit: byte offset of the vreg's row in a table of
// 64 16-bit entries per vreg), toggle[8] (32 bit: the width-w mask (1<<w)-1, or 0), test[8]
// (likewise), wl[8] (16 bit: 32 - width; the range straddles a 32-bit word iff
// (register & 31) > wl).  Ranges wider than 32 registers carry wl = 0x8000 | width and
// toggle, test as 0/1 flags.  A no-op names the spare vreg V with empty masks.
__device__ __forceinline__ void put_event(uint4 *ev, size_t idx, uint32_t v, uint32_t w, bool test, bool toggle)
{
    unsigned char *g = reinterpret_cast<unsigned char *>(ev) + (idx >> 3) * 112;
    const uint32_t slot = (uint32_t)(idx & 7);
    const uint32_t wm = w > 32 ? 1u : (w == 32 ? 0xFFFFFFFFu : ((1u << w) - 1u));
    reinterpret_cast<uint32_t *>(g)[slot] = v * 128u;
    reinterpret_cast<uint32_t *>(g + 32)[slot] = toggle ? wm : 0u;
    reinterpret_cast<uint32_t *>(g + 64)[slot] = test ? wm : 0u;
    reinterpret_cast<uint16_t *>(g + 96)[slot] = (uint16_t)(w > 32 ? (0x8000u | w) : (32u - w));
}

// Walk events of one chunk: entry occupancy (ascending vreg id), then per instruction the
// releases of dying reads, the definitions, and the releases of dead co-definitions.
__global__ void k_fill_events(const uint32_t *__restrict__ chunk_i0, const uint32_t *__restrict__ chunk_i1,
                              const uint32_t *__restrict__ op_off, const uint8_t *__restrict__ ndefs,
                              const uint32_t *__restrict__ op_vreg, const uint8_t *__restrict__ width,
                              const uint8_t *__restrict__ opflags, uint32_t Wv,
                              const uint32_t *__restrict__ chunk_entry, const uint32_t *__restrict__ centry_cnt,
                              const uint32_t *__restrict__ ev_off, const uint32_t *__restrict__ cev_off,
                              uint4 *ev, const uint32_t *__restrict__ chunk_blk, uint4 *el, uint32_t *el_count)
{
    __shared__ uint32_t s_scan[34];
    const uint32_t c = blockIdx.x;
    const size_t base = cev_off[c];
    uint32_t total;
    compact_bits(chunk_entry + (size_t)c * Wv, Wv, s_scan, &total, [&](uint32_t rank, uint32_t v) {
        put_event(ev, base + rank, v, width[v], true, true);
    });
    const uint32_t i0 = chunk_i0[c], i1 = chunk_i1[c];
    const uint32_t e_base = centry_cnt[c];
    for (uint32_t i = i0 + threadIdx.x; i < i1; i += NT) {
        uint32_t e = e_base + (ev_off[i] - ev_off[i0]);
        const uint32_t o0 = op_off[i], o1 = op_off[i + 1], nd = ndefs[i];
        for (uint32_t o = o0 + nd; o < o1; ++o)
            if (opflags[o] & OPF_KILL) {
                const uint32_t v = op_vreg[o];
                put_event(ev, base + (e++), v, width[v], false, true);
            }
        for (uint32_t o = o0; o < o0 + nd; ++o)
            if (!(opflags[o] & OPF_ELIDE)) {
                const uint32_t v = op_vreg[o];
                put_event(ev, base + (e++), v, width[v], true, (opflags[o] & OPF_SET) != 0);
            } else {  // no event: listed (in any order) for the recount of through-set collisions
                el[atomicAdd(el_count, 1u)] = make_uint4(i, c, op_vreg[o], chunk_blk[c]);
            }
        for (uint32_t o = o0; o < o0 + nd; ++o)
            if ((opflags[o] & OPF_POST) && !(opflags[o] & OPF_ELIDE)) {
                const uint32_t v = op_vreg[o];
                put_event(ev, base + (e++), v, width[v], false, true);
            }
    }
}

__global__ void k_fill_through(uint32_t Wv, const uint32_t *__restrict__ blk_th, const uint8_t *__restrict__ width,
                               const uint32_t *__restrict__ th_off, uint32_t *th)
{
    __shared__ uint32_t s_scan[34];
    const uint32_t b = blockIdx.x;
    const uint32_t base = th_off[b];
    uint32_t total;
    compact_bits(blk_th + (size_t)b * Wv, Wv, s_scan, &total,
                 [&](uint32_t rank, uint32_t v) { th[base + rank] = v | ((uint32_t)width[v] << 16); });
}

// First walk event of every chunk (each chunk padded to a multiple of 8 events), first through-set
// entry of every block, and both totals: totals[2] = events with padding, totals[3] = through entries.
// One thread block; the arrays are short (chunks, blocks).
// Also ls_adj[b] (see k_instr_walk) and totals[4] = length of all short live-after lists.
__global__ void k_offsets(uint32_t nC, uint32_t nB, const uint32_t *__restrict__ cev, const uint32_t *__restrict__ th_cnt,
                          uint32_t *cev_off, uint32_t *th_off, unsigned long long *totals,
                          const uint32_t *__restrict__ blk_off, uint32_t *ls_adj)
{
    __shared__ uint32_t s_scan[34];
    __shared__ unsigned long long s_carry;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    for (int which = 0; which < 2; ++which) {
        const uint32_t n = which == 0 ? nC : nB;
        const uint32_t *src = which == 0 ? cev : th_cnt;
        uint32_t *dst = which == 0 ? cev_off : th_off;
        for (uint32_t base = 0; base < n; base += NT) {
            const uint32_t i = base + threadIdx.x;
            uint32_t x = i < n ? src[i] : 0u;
            if (which == 0) x = (x + 7u) / 8u * 8u;
            uint32_t total;
            const uint32_t ex = block_excl_scan(x, s_scan, &total);
            const unsigned long long carry = s_carry;
            if (i < n) dst[i] = (uint32_t)(carry + ex);
            __syncthreads();
            if (threadIdx.x == 0) s_carry = carry + total;
            __syncthreads();
        }
        if (threadIdx.x == 0) {
            dst[n] = s_carry > 0xFFFFFFF0ull ? 0xFFFFFFF0u : (uint32_t)s_carry;
            totals[2 + which] = s_carry;
            s_carry = 0;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        unsigned long long pre = 0;  // through-set entries of all instructions of the blocks before b
        for (uint32_t b = 0; b < nB; ++b) {
            ls_adj[b] = (uint32_t)pre - blk_off[b] * th_cnt[b];
            pre += (unsigned long long)(blk_off[b + 1] - blk_off[b]) * th_cnt[b];
        }
        totals[4] = totals[0] - pre;
    }
}

// --------------------------------------------------------------------------- host
namespace {
template <typename T>
cudaError_t pool_get(VlArena &arena, T **out, size_t n)
{
    return arena.alloc((void **)out, std::max<size_t>(n, 1) * sizeof(T) + 64);
}
}  // namespace
#define KEEP(out, n) VL_CUDA(p, pool_get(p->live_arena, out, n))
#define TMP(out, n) VL_CUDA(p, pool_get(p->tmp_arena, out, n))
#define LAYOUT(out, n) VL_CUDA(p, pool_get(p->layout_arena, out, n))

static inline bool grid_nonempty(uint32_t g) { return g > 0; }
static inline bool grid_nonempty(dim3 g) { return g.x > 0 && g.y > 0 && g.z > 0; }
#define LAUNCH(kernel, grid, smem, st, ...)                          \
    do {                                                             \
        if (grid_nonempty(grid)) {                                   \
            kernel<<<(grid), NT, (smem), (st)>>>(__VA_ARGS__);       \
            g_vl_launches.fetch_add(1);                              \
        }                                                            \
    } while (0)

// Chunks, pieces and walk items depend on the program and on the chunk size only: they are laid
// out (and uploaded) when the chunk size changes, not on every call.
static int vl_layout(vl_program *p, cudaStream_t st)
{
    if (p->layout_chunk_instrs == p->chunk_instrs) return VL_OK;
    const uint32_t nB = p->nB;
    p->layout_chunk_instrs = 0;
    p->sizes_known = false;
    VL_CUDA(p, cudaDeviceSynchronize());  // earlier work (on any stream) may still read the old layout
    p->layout_arena.reset();
    p->tables_built = false;
    p->d_vreg16 = nullptr; p->d_slotmeta = nullptr; p->d_opoff = nullptr; p->d_first4 = nullptr;
    p->d_first_def_instr = nullptr; p->d_vinfo = nullptr;
    std::vector<uint32_t> c_i0, c_i1, c_blk, blk_c_off(nB + 1, 0), p_i0, p_i1, p_chunk, c_p_off;
    for (uint32_t b = 0; b < nB; ++b) {
        const uint64_t s = p->h_blk_off[b], n = p->h_blk_off[b + 1] - s;
        uint64_t nc = (n + p->chunk_instrs - 1) / p->chunk_instrs;
        // a walk item is shared by 8 warps, one chunk each at a time: a chunk count that is a multiple
        // of 8 keeps them equally busy (the chunks get a little shorter than asked for)
        if (nc > 4 && n >= 8 * 16) nc = (nc + 7) / 8 * 8;
        for (uint64_t j = 0; j < nc; ++j) {
            const uint32_t i0 = (uint32_t)(s + j * n / nc), i1 = (uint32_t)(s + (j + 1) * n / nc);
            c_p_off.push_back((uint32_t)p_i0.size());
            for (uint32_t q0 = i0; q0 < i1; q0 += PIECE_INSTRS) {
                p_i0.push_back(q0);
                p_i1.push_back(std::min(i1, q0 + PIECE_INSTRS));
                p_chunk.push_back((uint32_t)c_i0.size());
            }
            c_i0.push_back(i0);
            c_i1.push_back(i1);
            c_blk.push_back(b);
        }
        blk_c_off[b + 1] = (uint32_t)c_i0.size();
    }
    c_p_off.push_back((uint32_t)p_i0.size());
    const uint32_t nC = p->nC = (uint32_t)c_i0.size();
    p->nP = (uint32_t)p_i0.size();
    // walk work items: runs of at most VL_ITEM_CHUNKS chunks of one block
    std::vector<uint32_t> it_blk, it_c0, it_c1;
    for (uint32_t b = 0; b < nB; ++b)
        for (uint32_t c = blk_c_off[b]; c < blk_c_off[b + 1]; c += VL_ITEM_CHUNKS) {
            it_blk.push_back(b);
            it_c0.push_back(c);
            it_c1.push_back(std::min(c + VL_ITEM_CHUNKS, blk_c_off[b + 1]));
        }
    p->nItems = (uint32_t)it_blk.size();
    auto up = [&](uint32_t **dst, const std::vector<uint32_t> &v) -> int {
        LAYOUT(dst, v.size());
        if (!v.empty()) VL_CUDA(p, cudaMemcpy(*dst, v.data(), v.size() * 4, cudaMemcpyHostToDevice));
        return VL_OK;
    };
    int rc;
    if ((rc = up(&p->d_chunk_i0, c_i0)) || (rc = up(&p->d_chunk_i1, c_i1)) || (rc = up(&p->d_chunk_blk, c_blk)) ||
        (rc = up(&p->d_blk_chunk_off, blk_c_off)) || (rc = up(&p->d_piece_i0, p_i0)) || (rc = up(&p->d_piece_i1, p_i1)) ||
        (rc = up(&p->d_piece_chunk, p_chunk)) || (rc = up(&p->d_chunk_piece_off, c_p_off)) ||
        (rc = up(&p->d_item_blk, it_blk)) || (rc = up(&p->d_item_c0, it_c0)) || (rc = up(&p->d_item_c1, it_c1)))
        return rc;
    const uint32_t Wp = (p->P + p->wmax + 31) / 32 + 1;
    p->use_th = (nB <= 32 && (uint64_t)nB * VL_MAX_GROUP * Wp * 4 <= 24 * 1024) ? 1 : 0;
    p->layout_chunk_instrs = p->chunk_instrs;
    (void)nC;
    return VL_OK;
}

// Enqueues one complete liveness run on st (every kernel, the clears before them, the copy of the
// status word and the list lengths to pinned host memory behind them).  Without remembered list
// lengths it waits once in the middle to read them.
static int live_enqueue(vl_program *p, cudaStream_t st)
{
    vl_free_liveness(p);
    int rc = VL_OK;
    const uint32_t nB = p->nB, nI = p->nI, V = p->V, nO = p->nO, Wv = p->Wv, nC = p->nC, nP = p->nP;
    const size_t smem2 = (size_t)2 * Wv * 4;
    const size_t walk_smem = smem2 + (size_t)(2 * WALK_CAP_I + 1 + WALK_CAP_O) * 4 + WALK_CAP_I + 16;

    // ---- results and tables that do not depend on the list lengths
    KEEP(&p->d_blk_in, (size_t)2 * nB * Wv);  // live-in rows, then live-out rows
    p->d_blk_out = p->d_blk_in + (size_t)nB * Wv;
    KEEP(&p->d_lo_off, (size_t)nI + 1);
    KEEP(&p->d_opflags, (size_t)nO);
    // the operand tables of the verify kernels depend on the program alone: made by the first run, kept
    const bool make_tables = !p->tables_built;
    if (!p->d_opoff) {
        LAYOUT(&p->d_first_def_instr, (size_t)V);
        LAYOUT(&p->d_vreg16, (size_t)p->nOp8 + 8);
        LAYOUT(&p->d_slotmeta, (size_t)p->nOp8 / 8);
        LAYOUT(&p->d_first4, (size_t)p->nOpT / 4);
        LAYOUT(&p->d_vinfo, (size_t)V);
        LAYOUT(&p->d_opoff, (size_t)p->nOpT / 4);
    }
    KEEP(&p->d_iflags, (size_t)nI);
    KEEP(&p->d_cev_off, (size_t)nC + 1);
    KEEP(&p->d_th_off, (size_t)nB + 1);
    KEEP(&p->d_th_cnt, (size_t)nB);
    KEEP(&p->d_ls_adj, (size_t)nB);
    KEEP(&p->d_blk_th, (size_t)nB * Wv);
    KEEP(&p->d_el, (size_t)nO);  // at most one entry per definition
    KEEP(&p->d_el_count, 1);

    uint32_t *piece_use, *piece_def, *piece_end, *chunk_use, *chunk_def, *chunk_touch, *chunk_end, *chunk_entry;
    uint32_t *blk_use, *blk_def, *lo_cnt, *ev_cnt, *ev_off, *centry_cnt, *cev, *first_occ;
    uint32_t *const blk_th = p->d_blk_th, *const th_cnt = p->d_th_cnt;
    uint8_t *opmeta;
    unsigned long long *totals;
    TMP(&piece_use, (size_t)nP * Wv);
    TMP(&piece_def, (size_t)nP * Wv);
    TMP(&piece_end, (size_t)nP * Wv);
    TMP(&chunk_use, (size_t)nC * Wv);
    TMP(&chunk_def, (size_t)nC * Wv);
    TMP(&chunk_end, (size_t)nC * Wv);
    TMP(&chunk_entry, (size_t)nC * Wv);
    TMP(&blk_use, (size_t)nB * Wv);
    TMP(&blk_def, (size_t)nB * Wv);
    TMP(&lo_cnt, (size_t)nI + 1);
    TMP(&ev_cnt, (size_t)nI + 1);
    TMP(&ev_off, (size_t)nI + 1);
    TMP(&centry_cnt, (size_t)nC);
    TMP(&cev, (size_t)nC);
    first_occ = nullptr;
    opmeta = nullptr;
    if (make_tables) {
        TMP(&first_occ, (size_t)V);
        TMP(&opmeta, (size_t)nO);
    }
    TMP(&chunk_touch, (size_t)nC * Wv + 16);  // followed by the totals: one memset clears both
    totals = reinterpret_cast<unsigned long long *>(chunk_touch + (((size_t)nC * Wv + 1) & ~(size_t)1));
    // what has to start from a known value: the fixed point's sets, the touch sets (updated with
    // atomics), the totals, the status word, and the two "lowest index so far" arrays
    VL_CUDA(p, cudaMemsetAsync(p->d_blk_in, 0, (size_t)2 * nB * Wv * 4, st));
    VL_CUDA(p, cudaMemsetAsync(chunk_touch, 0, ((size_t)nC * Wv + 16) * 4, st));
    VL_CUDA(p, cudaMemsetAsync(p->d_status, 0, 4, st));
    VL_CUDA(p, cudaMemsetAsync(p->d_el_count, 0, 4, st));
    if (make_tables) {
        VL_CUDA(p, cudaMemsetAsync(first_occ, 0xFF, std::max<size_t>(V, 1) * 4, st));
        VL_CUDA(p, cudaMemsetAsync(p->d_first_def_instr, 0xFF, std::max<size_t>(V, 1) * 4, st));
    }

    LAUNCH(k_chunk_sets, nP, smem2, st, p->d_piece_i0, p->d_piece_i1, p->d_op_off, p->d_ndefs, p->d_op_vreg, Wv,
           piece_use, piece_def);
    const uint32_t wgrid = (Wv + NT - 1) / NT;
    if (nC) LAUNCH(k_block_sets, dim3(wgrid, nC), 0, st, p->d_chunk_piece_off, Wv, piece_use, piece_def, chunk_use, chunk_def);
    LAUNCH(k_block_sets, dim3(wgrid, nB), 0, st, p->d_blk_chunk_off, Wv, chunk_use, chunk_def, blk_use, blk_def);
    {
        const size_t fp_smem = ((size_t)4 * nB * NT + nB + 1 + p->nE) * 4;
        if (fp_smem <= 48 * 1024)
            LAUNCH(k_fixed_point<true>, wgrid, fp_smem, st, nB, p->nE, Wv, p->d_succ_off, p->d_succ, blk_use, blk_def,
                   p->d_blk_in, p->d_blk_out, p->d_status);
        else
            LAUNCH(k_fixed_point<false>, wgrid, 0, st, nB, p->nE, Wv, p->d_succ_off, p->d_succ, blk_use, blk_def,
                   p->d_blk_in, p->d_blk_out, p->d_status);
    }
    LAUNCH(k_chunk_boundaries, dim3(wgrid, nB), 0, st, p->d_blk_chunk_off, Wv, p->d_blk_out, chunk_use, chunk_def,
           chunk_end, chunk_entry);
    if (nC) LAUNCH(k_chunk_boundaries, dim3(wgrid, nC), 0, st, p->d_chunk_piece_off, Wv, chunk_end, piece_use, piece_def,
                   piece_end, (uint32_t *)nullptr);
    if (nP) k_instr_walk<false><<<nP, 32, walk_smem, st>>>(p->d_piece_i0, p->d_piece_i1, p->d_op_off, p->d_ndefs,
           p->d_op_vreg, Wv, piece_end, lo_cnt, ev_cnt, p->d_opflags, p->d_piece_chunk, chunk_touch,
           (const uint32_t *)nullptr, (uint32_t *)nullptr, (const uint32_t *)nullptr, (const uint32_t *)nullptr,
           (const uint32_t *)nullptr, (const uint32_t *)nullptr, (uint32_t *)nullptr);
    k_scan<<<2, 1024, 0, st>>>(lo_cnt, p->d_lo_off, ev_cnt, ev_off, nI, totals, p->d_status);
    g_vl_launches.fetch_add(nP ? 2 : 1);
    LAUNCH(k_block_through, dim3(wgrid, nB), 0, st, p->d_blk_chunk_off, Wv, p->use_th, p->d_blk_in, chunk_touch, blk_th);
    LAUNCH(k_chunk_entry, nC, 0, st, p->d_chunk_blk, p->d_chunk_i0, p->d_chunk_i1, Wv, blk_th, chunk_entry, ev_off,
           centry_cnt, cev);
    LAUNCH(k_row_popc, nB, 0, st, Wv, blk_th, th_cnt);
    k_offsets<<<1, NT, 0, st>>>(nC, nB, cev, th_cnt, p->d_cev_off, p->d_th_off, totals, p->d_blk_off, p->d_ls_adj);
    g_vl_launches.fetch_add(1);

    // ---- list lengths: read back on the first run with this layout; later runs allocate from the
    // lengths they remember (same program, same layout) and only compare at the end
    uint32_t status = 0;
    unsigned long long h_tot[5] = {0, 0, 0, 0, 0};
    if (!p->sizes_known) {
        VL_CUDA(p, cudaMemcpyAsync(&status, p->d_status, 4, cudaMemcpyDeviceToHost, st));
        VL_CUDA(p, cudaMemcpyAsync(h_tot, totals, 40, cudaMemcpyDeviceToHost, st));
        VL_CUDA(p, cudaStreamSynchronize(st));
        if (status & ST_NO_CONVERGE) return VL_ERR_NO_CONVERGE;
        if (status & ST_NOT_STRICT) return VL_ERR_NOT_STRICT;
        if (status & ST_SIZE_OVERFLOW) return VL_ERR_UNSUPPORTED;
        if (h_tot[2] > 0xFFFFFFF0ull) return VL_ERR_UNSUPPORTED;
        p->known_lo_len = h_tot[0];
        p->known_steps = h_tot[2];
        p->known_thn = h_tot[3];
        p->known_ls_len = h_tot[4];
    }
    p->lo_len = p->known_lo_len;
    const uint64_t steps = p->known_steps;  // walk events in total, every chunk padded to a multiple of 8 with no-ops
    p->ev_total = (uint32_t)steps;
    p->th_len = (uint32_t)p->known_thn;

    KEEP(&p->d_lo, (size_t)p->lo_len);
    KEEP(&p->d_ls, (size_t)p->known_ls_len);
    KEEP(&p->d_ev, (size_t)(steps / 8 + 2) * 7);  // two no-op groups behind the last chunk: the walk reads ahead
    KEEP(&p->d_th, (size_t)p->known_thn);
    LAUNCH(k_fill_noop, (uint32_t)std::min<uint64_t>(1024, (steps + NT - 1) / NT + 1), 0, st, p->d_ev,
           (size_t)(steps / 8 + 2), V);  // every slot starts as a no-op event

    // The list fill, the operand tables and the walk events do not depend on each other: the latter
    // two run on side streams beside the fill (as parallel branches when the run is recorded).
    cudaStream_t *lanes = nullptr;
    rc = vl_lane_streams(p, &lanes);
    if (rc != VL_OK) return rc;
    cudaStream_t sa = lanes[VL_LANES], sb = lanes[VL_LANES + 1];
    VL_CUDA(p, cudaEventRecord(p->ev_side[0], st));
    VL_CUDA(p, cudaStreamWaitEvent(sa, p->ev_side[0], 0));
    VL_CUDA(p, cudaStreamWaitEvent(sb, p->ev_side[0], 0));
    if (nP) k_instr_walk<true><<<nP, 32, walk_smem, st>>>(p->d_piece_i0, p->d_piece_i1, p->d_op_off, p->d_ndefs,
           p->d_op_vreg, Wv, piece_end, (uint32_t *)nullptr, (uint32_t *)nullptr, (uint8_t *)nullptr,
           (const uint32_t *)p->d_piece_chunk, (uint32_t *)nullptr, (const uint32_t *)p->d_lo_off, p->d_lo,
           (const uint32_t *)p->d_chunk_blk, (const uint32_t *)blk_th, (const uint32_t *)p->d_ls_adj,
           (const uint32_t *)th_cnt, p->d_ls);
    if (nP) g_vl_launches.fetch_add(1);
    if (make_tables) {
        LAUNCH(k_first_occ, (nI + NT - 1) / NT, 0, sa, nI, p->d_op_off, p->d_ndefs, p->d_op_vreg, first_occ,
               p->d_first_def_instr);
        LAUNCH(k_vreg_info, (V + NT - 1) / NT, 0, sa, V, p->d_width, first_occ, p->d_first_def_instr, p->d_vinfo);
        LAUNCH(k_operand_meta, (nI + NT - 1) / NT, 0, sa, nI, p->d_op_off, p->d_ndefs, p->d_op_vreg, first_occ,
               p->d_opflags, p->d_vreg16, opmeta, p->d_status);
        LAUNCH(k_pack_slots, (p->nOpT / 8 + NT - 1) / NT, 0, sa, nO, p->nOp8, p->nOpT / 8, V, opmeta, p->d_vreg16, p->d_slotmeta,
               p->d_opoff, p->d_first4);
    }
    LAUNCH(k_instr_flags, (nI + NT - 1) / NT, 0, sa, nI, p->d_op_off, p->d_ndefs, p->d_opflags, p->d_iflags);
    LAUNCH(k_fill_events, nC, 0, sb, p->d_chunk_i0, p->d_chunk_i1, p->d_op_off, p->d_ndefs, p->d_op_vreg, p->d_width,
           p->d_opflags, Wv, chunk_entry, centry_cnt, ev_off, p->d_cev_off, p->d_ev, p->d_chunk_blk, p->d_el,
           p->d_el_count);
    LAUNCH(k_fill_through, nB, 0, sb, Wv, blk_th, p->d_width, p->d_th_off, p->d_th);
    VL_CUDA(p, cudaEventRecord(p->ev_side[1], sa));
    VL_CUDA(p, cudaEventRecord(p->ev_side[2], sb));
    VL_CUDA(p, cudaStreamWaitEvent(st, p->ev_side[1], 0));
    VL_CUDA(p, cudaStreamWaitEvent(st, p->ev_side[2], 0));
    p->bank_fast = ((p->B == 1 || p->B == 2 || p->B == 4) && !p->bank_many) ? 1 : 0;
    VL_CUDA(p, cudaMemcpyAsync(p->h_live, p->d_status, 4, cudaMemcpyDeviceToHost, st));
    VL_CUDA(p, cudaMemcpyAsync(p->h_live + 2, totals, 40, cudaMemcpyDeviceToHost, st));
    p->tables_built = true;
    return rc;
}

// A run is the same sequence of launches with the same arguments every time once the layout and
// the list lengths are settled (the pools hand out the same addresses after a rewind).  The third
// run with settled lengths is therefore recorded as a CUDA graph while it is enqueued, and later
// runs replay the graph: one launch call instead of about thirty, which is what small programs and
// batches of programs spend their time on.  Everything is recomputed on the device on every run.
int vl_liveness_impl(vl_program *p, cudaStream_t st)
{
    vl_live_settle(p);  // the pinned words of an earlier run are about to be reused
    int rc = vl_layout(p, st);
    if (rc != VL_OK) return rc;
    if (!p->h_live) VL_CUDA(p, cudaHostAlloc((void **)&p->h_live, 64, cudaHostAllocDefault));
    if (!p->ev_live) VL_CUDA(p, cudaEventCreateWithFlags(&p->ev_live, cudaEventDisableTiming));
    if (!p->sizes_known) vl_drop_live_graph(p);
    bool replayed = false;
    if (p->sizes_known && p->live_graph) {
        if (cudaGraphLaunch(p->live_graph, st) == cudaSuccess) {
            g_vl_launches.fetch_add(p->live_graph_launches);
            replayed = true;
        } else {
            cudaGetLastError();
            vl_drop_live_graph(p);
        }
    }
    if (!replayed) {
        bool capturing = false;
        cudaStream_t rec = st;
        if (p->sizes_known && p->graph_opt && ++p->settled_runs >= 2) {
            // recorded on an internal stream (the caller's may be the legacy default stream, which
            // cannot record; nothing runs while recording), then launched on the caller's
            cudaStream_t *lanes = nullptr;
            if (vl_lane_streams(p, &lanes) == VL_OK) {
                rec = lanes[0];
                capturing = cudaStreamBeginCapture(rec, cudaStreamCaptureModeThreadLocal) == cudaSuccess;
            }
            if (!capturing) { cudaGetLastError(); p->graph_opt = 0; rec = st; }
        }
        const uint64_t launches0 = g_vl_launches.load();
        rc = live_enqueue(p, rec);
        if (capturing) {
            cudaGraph_t graph = nullptr;
            cudaError_t e = cudaStreamEndCapture(rec, &graph);
            if (e == cudaSuccess && rc == VL_OK) e = cudaGraphInstantiate(&p->live_graph, graph, 0);
            if (graph) cudaGraphDestroy(graph);
            if (e != cudaSuccess || rc != VL_OK) {
                cudaGetLastError();
                vl_drop_live_graph(p);
                p->graph_opt = 0;  // recording does not work here: enqueue directly from now on
                if (rc == VL_OK) rc = live_enqueue(p, st);
            } else {
                p->live_graph_launches = g_vl_launches.load() - launches0;
                VL_CUDA(p, cudaGraphLaunch(p->live_graph, st));  // what was recorded has not run yet
            }
        }
        if (rc != VL_OK) return rc;
    }
    VL_CUDA(p, cudaEventRecord(p->ev_live, st));
    VL_CUDA(p, cudaGetLastError());
    p->live_pending = true;
    p->live_ok = true;
    if (p->sizes_known) return VL_OK;  // lengths remembered from an earlier run: checked when the results are used
    rc = vl_live_settle(p);
    if (rc == VL_OK) { p->sizes_known = true; p->settled_runs = 0; }
    return rc;
}

void vl_drop_live_graph(vl_program *p)
{
    if (p->live_graph) cudaGraphExecDestroy(p->live_graph);
    p->live_graph = nullptr;
    p->settled_runs = 0;
}

int vl_live_settle(vl_program *p)
{
    if (!p->live_pending) return VL_OK;
    p->live_pending = false;
    p->live_ok = false;
    VL_CUDA(p, cudaEventSynchronize(p->ev_live));
    const uint32_t status = p->h_live[0];
    unsigned long long h_tot[5];
    memcpy(h_tot, p->h_live + 2, 40);
    if (status & ST_NO_CONVERGE) return VL_ERR_NO_CONVERGE;
    if (status & ST_NOT_STRICT) return VL_ERR_NOT_STRICT;
    if (status & ST_SIZE_OVERFLOW) return VL_ERR_UNSUPPORTED;
    if (h_tot[0] != p->known_lo_len || h_tot[2] != p->known_steps || h_tot[3] != p->known_thn ||
        h_tot[4] != p->known_ls_len) {
        // the lengths the run allocated from do not fit what it computed: the next run measures again
        p->sizes_known = false;
        return VL_ERR_CUDA;
    }
    p->live_ok = true;
    return VL_OK;
}
