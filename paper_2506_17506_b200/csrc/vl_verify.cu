// The verify kernel: G candidates per thread block, packed side by side.
//
// Pass 1 streams the G candidate rows (bulk async copies into a shared-memory ring, completion
// on mbarriers), builds the vreg -> preg tables T (G 16-bit entries per vreg, shared memory)
// from first occurrences and compares every other occurrence with T (Consistency).
// One sweep over the vregs checks [T, T+width) against the register file (Realizability).
// A sweep over the instructions with two or more distinct sources tallies bank conflicts from T.
// Pass 2 walks the program's precompiled event stream, one thread per chunk of instructions,
// keeping a bitmask of occupied registers per (chunk, candidate) in shared memory (Safety).
// A chunk whose walk sees no collision provably has no overlap; chunks that do are recounted
// exactly from the per-instruction live-after lists by whole warps.
#include <algorithm>

#include "vl_internal.cuh"

#define MAX_STAGES 4
#define WU 8  // walk events fetched per batch

struct VParams {
    uint32_t nI, V, nO, nOp8, P, B, Bmask, nB, nC, nGroups, Wp, ntiles;
    int bank_fast, use_th;
    const uint16_t *vreg16;
    const uint64_t *slotmeta;
    const uint32_t *vinfo, *first_def_instr, *th_off, *th, *grp_off, *ev;
    const uint32_t *chunk_i0, *chunk_i1, *chunk_blk, *op_off, *op_vreg, *lo_off, *lo;
    const uint8_t *ndefs, *width, *opflags;
    const uint2 *bank_list;
    uint32_t bank_seg[4];  // entries with n = 2, 3, 4 distinct sources: [seg[n-2], seg[n-1])
    const uint16_t *cand;
    uint64_t K, pitch;
    vl_verdict *out;
    uint32_t *status;
    uint32_t S, NS, AW;
    uint32_t off_T, off_region, off_occ, off_anom, off_misc;
};

struct Misc {
    unsigned long long bar[MAX_STAGES];
    uint32_t flags[VL_MAX_GROUP], minop[VL_MAX_GROUP], minR[VL_MAX_GROUP], minD[VL_MAX_GROUP];
    uint32_t pairs[VL_MAX_GROUP], bank[VL_MAX_GROUP], nout[VL_MAX_GROUP], out_v[VL_MAX_GROUP];
    uint32_t out_raw[VL_MAX_GROUP], full[VL_MAX_GROUP], ganom[VL_MAX_GROUP], thcol[VL_MAX_GROUP];
    uint32_t abort_flag, any_anom;
};

// Optional per-phase cycle counters (thread 0 of every block adds its elapsed clocks to
// status[2 + phase]); compiled in only with -DVL_PHASE_TIMERS, for profiling builds.
#ifdef VL_PHASE_TIMERS
#define PT_INIT() long long pt_last = clock64()
#define PT(idx)                                                                \
    do {                                                                       \
        if (threadIdx.x == 0) {                                                \
            long long now = clock64();                                         \
            atomicAdd(q.status + 2 + (idx), (uint32_t)((now - pt_last) >> 6)); \
            pt_last = now;                                                     \
        }                                                                      \
    } while (0)
#else
#define PT_INIT()
#define PT(idx)
#endif

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

// ------------------------------------------------------------- packed table access
// T holds, per vreg, the G candidates' registers side by side (16 bits each).
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

// One walk event of one candidate, any width, on a mask whose consecutive 32-bit words are `stride`
// words apart.  tm: all ones if the event tests, xm: all ones if it toggles occupancy (becoming
// occupied and being released are both a toggle as long as no collision has been seen; after a
// collision the chunk is recounted exactly anyway).  [t, t+w) lies inside the mask.
__device__ __forceinline__ uint32_t occ_event_wide(uint32_t *mask, uint32_t stride, uint32_t t, uint32_t w, uint32_t tm,
                                                   uint32_t xm)
{
    uint32_t viol = 0, left = w, pos = t;
    while (left) {
        const uint32_t s2 = pos & 31, n = min(left, 32 - s2);
        const uint32_t m = (n == 32 ? 0xFFFFFFFFu : ((1u << n) - 1u)) << s2;
        uint32_t *a = mask + (pos >> 5) * stride;
        const uint32_t o = *a;
        viol |= o & m & tm;
        *a = o ^ (m & xm);
        pos += n;
        left -= n;
    }
    return viol;
}

// ------------------------------------------------------------------------- kernel
template <int G, int NT, bool WIDE>
__global__ void __launch_bounds__(NT) k_verify(const VParams q)
{
    constexpr uint32_t TILE = NT * 8;  // operands per tile and candidate
    constexpr uint32_t STAGE_BYTES = TILE * 2;
    extern __shared__ __align__(16) unsigned char smem[];
    uint16_t *Tt = reinterpret_cast<uint16_t *>(smem + q.off_T);
    unsigned char *region = smem + q.off_region;
    uint32_t *s_th = reinterpret_cast<uint32_t *>(region);             // [nB][G][Wp], pass 2 only
    uint32_t *s_occ = reinterpret_cast<uint32_t *>(smem + q.off_occ);  // [Wp][G][S], pass 2 only
    uint32_t *s_anom = reinterpret_cast<uint32_t *>(smem + q.off_anom);
    Misc *M = reinterpret_cast<Misc *>(smem + q.off_misc);

    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint64_t k0 = (uint64_t)blockIdx.x * G;
    const uint16_t *rows[G];
#pragma unroll
    for (int g = 0; g < G; ++g) rows[g] = q.cand + min(k0 + g, q.K - 1) * q.pitch;

    if (tid < G) {
        M->flags[tid] = 0; M->minop[tid] = 0xFFFFFFFFu; M->minR[tid] = 0xFFFFFFFFu; M->minD[tid] = 0xFFFFFFFFu;
        M->pairs[tid] = 0; M->bank[tid] = 0; M->nout[tid] = 0; M->out_v[tid] = 0; M->out_raw[tid] = 0;
        M->full[tid] = 0; M->ganom[tid] = 0; M->thcol[tid] = 0;
    }
    if (tid == 0) {
        M->abort_flag = 0;
        M->any_anom = 0;
        for (uint32_t s = 0; s < q.NS; ++s) mbar_init(&M->bar[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (uint32_t i = tid; i < G * q.AW; i += NT) s_anom[i] = 0;
    __syncthreads();
    PT_INIT();

    // ---------------------------------------------------------------- pass 1
    auto issue_tile = [&](uint32_t t) {
        const uint32_t stage = t % q.NS;
        const uint32_t bytes = min(TILE, q.nOp8 - t * TILE) * 2;
        mbar_expect_tx(&M->bar[stage], bytes * G);
#pragma unroll
        for (int g = 0; g < G; ++g)
            bulk_g2s(region + (size_t)(stage * G + g) * STAGE_BYTES, rows[g] + (size_t)t * TILE, bytes, &M->bar[stage]);
    };
    if (tid == 0)
        for (uint32_t t = 0; t < q.NS && t < q.ntiles; ++t) issue_tile(t);

    // operand metadata of the next tile is fetched one iteration ahead (global memory, L2 latency)
    uint4 nx_v4 = make_uint4(0, 0, 0, 0);
    uint32_t nx_first = 0;
    if (tid * 8 < q.nOp8) {
        nx_v4 = *reinterpret_cast<const uint4 *>(q.vreg16 + tid * 8);
        nx_first = (uint32_t)q.slotmeta[tid] & 0xFFu;
    }
    for (uint32_t t = 0; t < q.ntiles; ++t) {
        const uint32_t stage = t % q.NS, parity = (t / q.NS) & 1;
        const uint4 v4 = nx_v4;
        const uint32_t first = nx_first;
        {
            const uint32_t o_next = (t + 1) * TILE + tid * 8;
            if (t + 1 < q.ntiles && o_next < q.nOp8) {
                nx_v4 = *reinterpret_cast<const uint4 *>(q.vreg16 + o_next);
                nx_first = (uint32_t)q.slotmeta[o_next >> 3] & 0xFFu;
            }
        }
        {  // bounded wait for the tile
            uint32_t spins = 0;
            const uint32_t limit = *(volatile uint32_t *)&M->abort_flag ? 64u : (1u << 22);
            while (!mbar_try_wait(&M->bar[stage], parity)) {
                if (++spins > limit) {
                    M->abort_flag = 1;
                    atomicOr(q.status, ST_DEVICE_WAIT);
                    break;
                }
            }
        }
        const uint32_t o_base = t * TILE + tid * 8;
        const bool act = o_base < q.nOp8;
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
        uint64_t pc[8];
        uint32_t vj[8];
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
        // first occurrences write the table ...
        if (act) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if ((first >> j) & 1) t_store<G>(Tt, vj[j], pc[j]);
        }
        __syncthreads();
        // the stage just read is free again: refill it with the tile NS ahead
        if (tid == 0 && t + q.NS < q.ntiles) issue_tile(t + q.NS);
        // ... and every occurrence is compared with it (a first occurrence trivially matches;
        // padding operands beyond n_operands are left out)
        if (act) {
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
        }
    }
    __syncthreads();
    PT(0);

    // ------------------------------------------------- realizability, one sweep over the vregs
    for (uint32_t v0 = tid; v0 < q.V; v0 += 4 * NT) {
        uint32_t vis[4], fds[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t v = v0 + u * NT;
            vis[u] = v < q.V ? q.vinfo[v] : 0u;
            fds[u] = v < q.V ? q.first_def_instr[v] : 0xFFFFFFFFu;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t v = v0 + u * NT, vi = vis[u];
            if (!(vi & VINFO_OCCURS)) continue;
            const uint32_t w = vi & 0xFFu;
            const uint64_t tt = t_load<G>(Tt, v);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const uint32_t tv = pk_get(tt, g);
                if (tv + w > q.P) {
                    if (vi & VINFO_DEFINED) {
                        atomicOr(&M->flags[g], (uint32_t)VL_OUT_OF_RANGE);
                        atomicMin(&M->minR[g], fds[u]);
                    }
                    if (atomicAdd(&M->nout[g], 1u) == 0) { M->out_v[g] = v; M->out_raw[g] = tv; }
                }
            }
        }
    }
    PT(1);

    // ------------------------------- bank tally from T: instructions with 2..4 distinct sources.
    // Distinct vregs read by one instruction are live together, so a candidate whose walk sees no
    // collision has them on distinct registers and only the banks need comparing; candidates with
    // a collision get the general tally further down.
    if (q.bank_fast) {
        constexpr uint64_t L1 = 0x0001000100010001ull;
        const uint64_t BM = L1 * q.Bmask;
        uint64_t acc = 0;
        auto same = [&](uint64_t x) -> uint64_t { return ((x | (x >> 1)) & L1) ^ L1; };  // per lane: x == 0
        for (uint32_t e = q.bank_seg[0] + tid; e < q.bank_seg[1]; e += NT) {
            const uint2 ids = q.bank_list[e];
            const uint64_t a = t_load<G>(Tt, ids.x & 0xFFFFu) & BM, b = t_load<G>(Tt, ids.x >> 16) & BM;
            acc += same(a ^ b);
        }
        for (uint32_t e = q.bank_seg[1] + tid; e < q.bank_seg[2]; e += NT) {
            const uint2 ids = q.bank_list[e];
            const uint64_t a = t_load<G>(Tt, ids.x & 0xFFFFu) & BM, b = t_load<G>(Tt, ids.x >> 16) & BM,
                           c = t_load<G>(Tt, ids.y & 0xFFFFu) & BM;
            acc += same(a ^ b) + (same(c ^ a) | same(c ^ b));
        }
        for (uint32_t e = q.bank_seg[2] + tid; e < q.bank_seg[3]; e += NT) {
            const uint2 ids = q.bank_list[e];
            const uint64_t a = t_load<G>(Tt, ids.x & 0xFFFFu) & BM, b = t_load<G>(Tt, ids.x >> 16) & BM,
                           c = t_load<G>(Tt, ids.y & 0xFFFFu) & BM, d = t_load<G>(Tt, ids.y >> 16) & BM;
            acc += same(a ^ b) + (same(c ^ a) | same(c ^ b)) + (same(d ^ a) | same(d ^ b) | same(d ^ c));
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            uint32_t x = pk_get(acc, g);
#pragma unroll
            for (int d = 16; d; d >>= 1) x += __shfl_xor_sync(0xffffffffu, x, d);
            if (lane == 0 && x) atomicAdd(&M->bank[g], x);
        }
    }
    __syncthreads();
    PT(2);
    // One vreg sticking out of the file cannot overlap another one out there: park it at P (bits
    // beyond P are padding) and walk as usual.  Two or more: that candidate is recounted in full.
    if (tid < G) {
        const uint32_t g = tid;
        if (M->nout[g] == 1) {
            if (M->out_raw[g] >= q.P) Tt[(size_t)M->out_v[g] * G + g] = (uint16_t)q.P;
        } else if (M->nout[g] >= 2) {
            M->full[g] = 1;
        }
        Tt[(size_t)q.V * G + g] = 0;  // the spare entry that no-op events look up
    }
    if (q.use_th)
        for (uint32_t i = tid; i < q.nB * G * q.Wp; i += NT) s_th[i] = 0;
    __syncthreads();

    // ---------------------------------------------------------------- pass 2
    // masks of the vregs that stay occupied through a whole block, per (block, candidate)
    if (q.use_th) {
        for (uint32_t b = 0; b < q.nB; ++b)
            for (uint32_t e = q.th_off[b] + tid; e < q.th_off[b + 1]; e += NT) {
                const uint32_t x = q.th[e], v = x & 0xFFFFu, w = x >> 16;
                const uint64_t tt = t_load<G>(Tt, v);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    if (M->full[g]) continue;
                    uint32_t pos = pk_get(tt, g), left = w;
                    while (left) {
                        const uint32_t s2 = pos & 31, n = min(left, 32 - s2);
                        const uint32_t m = (n == 32 ? 0xFFFFFFFFu : ((1u << n) - 1u)) << s2;
                        const uint32_t old = atomicOr(&s_th[(size_t)(b * G + g) * q.Wp + (pos >> 5)], m);
                        if (old & m) atomicOr(&M->thcol[g], 1u << b);  // through-sets are used only if nB <= 32
                        pos += n;
                        left -= n;
                    }
                }
            }
        __syncthreads();
    }
    uint32_t fullmask = 0;
#pragma unroll
    for (int g = 0; g < G; ++g) fullmask |= M->full[g] ? (1u << g) : 0u;
    PT(3);

    if (tid < q.S) {
        const uint32_t stride = G * q.S;  // words between consecutive mask words of one (slot, candidate)
        const uint32_t nop = q.V | (1u << 16);
        uint32_t tsel[G];  // a candidate that is recounted in full is walked on register 0 (its table may hold anything)
#pragma unroll
        for (int g = 0; g < G; ++g) tsel[g] = (fullmask & (1u << g)) ? 0u : 0xFFFFu;
        for (uint32_t gi = warp; gi < q.nGroups; gi += q.S / 32) {
            const uint32_t c = gi * 32 + lane;
            const bool have = c < q.nC;
            const uint32_t b = have ? q.chunk_blk[c] : 0;
            for (uint32_t wd = 0; wd < q.Wp; ++wd)
#pragma unroll
                for (int g = 0; g < G; ++g)
                    s_occ[(size_t)(wd * G + g) * q.S + tid] =
                        (q.use_th && have) ? s_th[(size_t)(b * G + g) * q.Wp + wd] : 0u;
            uint32_t viol[G];
#pragma unroll
            for (int g = 0; g < G; ++g) viol[g] = 0;
            const uint32_t s0 = q.grp_off[gi], s1 = q.grp_off[gi + 1];
            uint32_t nxt[WU];
#pragma unroll
            for (int u = 0; u < WU; ++u) nxt[u] = (s0 + u < s1) ? q.ev[(size_t)(s0 + u) * 32 + lane] : nop;
            for (uint32_t s = s0; s < s1; s += WU) {
                uint32_t cur[WU];
                uint64_t tts[WU];
#pragma unroll
                for (int u = 0; u < WU; ++u) cur[u] = nxt[u];
#pragma unroll
                for (int u = 0; u < WU; ++u)
                    nxt[u] = (s + WU + u < s1) ? q.ev[(size_t)(s + WU + u) * 32 + lane] : nop;
#pragma unroll
                for (int u = 0; u < WU; ++u) tts[u] = t_load<G>(Tt, cur[u] & 0xFFFFu);
#pragma unroll
                for (int u = 0; u < WU; ++u) {
                    const uint32_t e = cur[u];
                    const uint32_t w = (e >> 16) & 0xFFu;
                    const uint32_t wm = (!WIDE || w < 32) ? ((1u << (w & 31)) - 1u) : 0xFFFFFFFFu;
                    const uint32_t tm = 0u - ((e >> 24) & 1u);
                    const uint32_t xm = (e & (EV_SET | EV_CLEAR)) ? 0xFFFFFFFFu : 0u;
                    if (!WIDE || w <= 32) {
                        // the G candidates' words are independent: all loads first, then all stores
                        uint32_t *a[G];
                        uint32_t o[G], m0[G], m1[G];
#pragma unroll
                        for (int g = 0; g < G; ++g) {
                            const uint32_t t = (uint32_t)(tts[u] >> (16 * g)) & tsel[g];
                            m0[g] = wm << (t & 31);
                            m1[g] = __funnelshift_l(wm, 0u, t);  // bits that spill into the next word
                            a[g] = s_occ + (size_t)g * q.S + tid + (t >> 5) * stride;
                            o[g] = *a[g];
                        }
                        uint32_t spill = 0;
#pragma unroll
                        for (int g = 0; g < G; ++g) {
                            if (fullmask & (1u << g)) continue;
                            viol[g] |= o[g] & m0[g] & tm;
                            *a[g] = o[g] ^ (m0[g] & xm);
                            spill |= m1[g];
                        }
                        if (spill) {
#pragma unroll
                            for (int g = 0; g < G; ++g) {
                                if (!m1[g] || (fullmask & (1u << g))) continue;
                                uint32_t *a2 = a[g] + stride;
                                const uint32_t o2 = *a2;
                                viol[g] |= o2 & m1[g] & tm;
                                *a2 = o2 ^ (m1[g] & xm);
                            }
                        }
                    } else {
#pragma unroll
                        for (int g = 0; g < G; ++g) {
                            if (fullmask & (1u << g)) continue;
                            viol[g] |= occ_event_wide(s_occ + (size_t)g * q.S + tid, stride, pk_get(tts[u], g), w, tm, xm);
                        }
                    }
                }
            }
            if (have) {
#pragma unroll
                for (int g = 0; g < G; ++g)
                    if (viol[g]) {
                        atomicOr(&s_anom[g * q.AW + (c >> 5)], 1u << (c & 31));
                        M->ganom[g] = 1;
                        M->any_anom = 1;
                    }
            }
        }
    }
    __syncthreads();
    PT(4);

    // ------------------------------------------- exact recount where the walk cannot vouch
    if (tid < G) {
        if (M->nout[tid] == 1) Tt[(size_t)M->out_v[tid] * G + tid] = (uint16_t)M->out_raw[tid];  // true value back
        if (M->full[tid] || M->thcol[tid]) { M->ganom[tid] = 1; M->any_anom = 1; }
    }
    __syncthreads();
    if (M->any_anom) {
        for (uint32_t item = 0; item < G * q.nC; ++item) {
            const uint32_t g = item / q.nC, c = item % q.nC;
            // a chunk that collided (or a candidate with several out-of-file vregs): every definition;
            // a block whose through-set collided: the definitions the walk skipped (a vreg redefined
            // from itself while it stays occupied), since everything else in it was walked exactly
            const bool all_defs = M->full[g] || ((s_anom[g * q.AW + (c >> 5)] >> (c & 31)) & 1u);
            const bool elided_only = !all_defs && ((M->thcol[g] >> (q.chunk_blk[c] & 31)) & 1u);
            if (!all_defs && !elided_only) continue;
            uint32_t pairs = 0, mind = 0xFFFFFFFFu;
            for (uint32_t i = q.chunk_i0[c] + warp; i < q.chunk_i1[c]; i += NT / 32) {
                const uint32_t o0 = q.op_off[i], nd = q.ndefs[i];
                const uint32_t l0 = q.lo_off[i], l1 = q.lo_off[i + 1];
                for (uint32_t d = o0; d < o0 + nd; ++d) {
                    if (elided_only && !(q.opflags[d] & OPF_ELIDE)) continue;
                    const uint32_t v = q.op_vreg[d];
                    const uint32_t s = Tt[(size_t)v * G + g], w = q.width[v];
                    uint32_t cnt = 0;
                    for (uint32_t e0 = l0; e0 < l1; e0 += 128) {  // 4 list entries per lane in flight
                        uint32_t us[4], ws[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const uint32_t e = e0 + u * 32 + lane;
                            us[u] = e < l1 ? q.lo[e] : v;
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u) ws[u] = q.vinfo[us[u]] & 0xFFu;
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            if (us[u] != v && ranges_overlap(s, w, Tt[(size_t)us[u] * G + g], ws[u])) ++cnt;
                    }
                    // co-defined vregs that are not live after the instruction
                    for (uint32_t d2 = o0 + lane; d2 < o0 + nd; d2 += 32) {
                        if (d2 == d || !(q.opflags[d2] & OPF_DEAD)) continue;
                        const uint32_t u = q.op_vreg[d2];
                        if (ranges_overlap(s, w, Tt[(size_t)u * G + g], q.width[u])) ++cnt;
                    }
#pragma unroll
                    for (int dd = 16; dd; dd >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, dd);
                    if (cnt) { pairs += cnt; mind = min(mind, i); }
                }
            }
            if (lane == 0 && pairs) {
                atomicAdd(&M->pairs[g], pairs);
                atomicMin(&M->minD[g], mind);
            }
        }
    }
    __syncthreads();
    PT(5);
    // ------------------- general bank tally (distinct registers, not distinct vregs) where needed
    uint32_t need_bank = 0;
#pragma unroll
    for (int g = 0; g < G; ++g)
        if (!q.bank_fast || M->ganom[g]) need_bank |= 1u << g;
    __syncthreads();
    if (need_bank) {
        if (tid < G && (need_bank >> tid) & 1u) M->bank[tid] = 0;
        __syncthreads();
        uint32_t bt[G];
#pragma unroll
        for (int g = 0; g < G; ++g) bt[g] = 0;
        for (uint32_t i = tid; i < q.nI; i += NT) {
            const uint32_t u0 = q.op_off[i] + q.ndefs[i], u1 = q.op_off[i + 1];
            for (uint32_t a = u0 + 1; a < u1; ++a) {
                const uint64_t ta = t_load<G>(Tt, q.op_vreg[a]);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    if (!((need_bank >> g) & 1u)) continue;
                    const uint32_t xa = pk_get(ta, g);
                    bool seen_value = false, seen_bank = false;
                    for (uint32_t bb = u0; bb < a; ++bb) {
                        const uint32_t xb = Tt[(size_t)q.op_vreg[bb] * G + g];
                        seen_value |= (xb == xa);
                        seen_bank |= (xb % q.B == xa % q.B);
                    }
                    // a new distinct register landing in a bank already in use costs one cycle
                    if (!seen_value && seen_bank) ++bt[g];
                }
            }
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            uint32_t x = bt[g];
#pragma unroll
            for (int d = 16; d; d >>= 1) x += __shfl_xor_sync(0xffffffffu, x, d);
            if (lane == 0 && x) atomicAdd(&M->bank[g], x);
        }
    }
    __syncthreads();
    PT(6);

    // ----------------------------------------------------------------- verdicts
    if (tid < G && k0 + tid < q.K) {
        const uint32_t g = tid;
        uint32_t first = 0xFFFFFFFFu;
        if (M->minop[g] != 0xFFFFFFFFu) {  // operand -> instruction: last i with op_off[i] <= operand
            const uint32_t o = M->minop[g];
            uint32_t lo_i = 0, hi_i = q.nI;  // invariant: op_off[lo_i] <= o < op_off[hi_i]
            while (hi_i - lo_i > 1) {
                const uint32_t mid = (lo_i + hi_i) >> 1;
                if (q.op_off[mid] <= o) lo_i = mid; else hi_i = mid;
            }
            first = lo_i;
        }
        first = min(first, min(M->minR[g], M->minD[g]));
        uint32_t flags = M->flags[g] | (M->pairs[g] ? (uint32_t)VL_INTERFERENCE : 0u);
        if (!flags) flags = VL_PASS;
        vl_verdict vd;
        vd.flags = flags;
        vd.first_violation_instr = first == 0xFFFFFFFFu ? -1 : (int32_t)first;
        vd.conflict_pairs = M->pairs[g];
        vd.bank_conflicts = M->bank[g];
        q.out[k0 + g] = vd;
    }
}

// --------------------------------------------------------------------------- host
namespace {
struct Plan { uint32_t G, NT, S, NS, smem, off_T, off_region, off_occ, off_anom, off_misc, AW, Wp; bool ok; };

inline uint64_t align16(uint64_t x) { return (x + 15u) & ~15ull; }

// Shared memory of one block: [T][region][anomaly bitmap][misc]; the region holds the copy ring in
// pass 1 and the through-set masks followed by the walkers' masks in pass 2.
Plan make_plan(const vl_program *p, uint32_t G, uint32_t NT, uint32_t budget, uint32_t min_slots)
{
    Plan pl{};
    pl.G = G; pl.NT = NT;
    pl.Wp = (p->P + p->wmax + 31) / 32;
    pl.AW = std::max(1u, (p->nC + 31) / 32);
    const uint64_t stage = (uint64_t)NT * 8 * 2 * G;
    const uint64_t tbytes = align16((uint64_t)(p->V + 1) * G * 2);
    const uint64_t thbytes = p->use_th ? align16((uint64_t)p->nB * G * pl.Wp * 4) : 0;
    const uint64_t anom = align16((uint64_t)G * pl.AW * 4);
    const uint64_t misc = align16(sizeof(Misc));
    const uint64_t fixed = tbytes + anom + misc;
    const uint64_t slot = (uint64_t)G * pl.Wp * 4;
    pl.ok = false;
    if (fixed + 2 * stage > budget || fixed + thbytes + 32 * slot > budget) return pl;
    const uint64_t room = budget - fixed;
    uint32_t S = (uint32_t)std::min<uint64_t>(NT, (room - thbytes) / slot) / 32 * 32;
    const uint32_t want = std::min<uint32_t>(NT, std::max(1u, p->nGroups) * 32);
    S = std::min(S, want);
    if (S < std::min(min_slots, want)) return pl;
    const uint32_t NS = (uint32_t)std::min<uint64_t>(MAX_STAGES, room / stage);
    const uint64_t region = std::max<uint64_t>((uint64_t)NS * stage, thbytes + (uint64_t)S * slot);
    pl.S = S; pl.NS = NS;
    pl.off_T = 0;
    pl.off_region = (uint32_t)tbytes;
    pl.off_occ = (uint32_t)(tbytes + thbytes);
    pl.off_anom = (uint32_t)(tbytes + align16(region));
    pl.off_misc = pl.off_anom + (uint32_t)anom;
    pl.smem = pl.off_misc + (uint32_t)misc;
    pl.ok = pl.smem <= budget;
    return pl;
}

template <int G, int NT, bool WIDE>
cudaError_t launch(const VParams &q, uint32_t grid, uint32_t smem, cudaStream_t st)
{
    cudaError_t e = cudaFuncSetAttribute(k_verify<G, NT, WIDE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_verify<G, NT, WIDE><<<grid, NT, smem, st>>>(q);
    return cudaGetLastError();
}
template <int G, int NT>
cudaError_t launch_w(bool wide, const VParams &q, uint32_t grid, uint32_t smem, cudaStream_t st)
{
    return wide ? launch<G, NT, true>(q, grid, smem, st) : launch<G, NT, false>(q, grid, smem, st);
}
}  // namespace

int vl_verify_impl(const vl_program *p, const uint16_t *d_cand, uint64_t K, uint64_t pitch, vl_verdict *d_out,
                   cudaStream_t st)
{
    const uint32_t SM_BYTES = 227 * 1024;
    // preference: the largest group that still lets two blocks share an SM, then anything that fits
    Plan pl{};
    const uint32_t groups[3] = {4, 2, 1};
    const uint32_t NT = p->threads_opt ? p->threads_opt : 256;
    for (int pass = 0; pass < 2 && !pl.ok; ++pass)
        for (uint32_t G : groups) {
            if (p->group_opt && G != p->group_opt) continue;
            const uint32_t budget = pass == 0 ? (SM_BYTES / 2 - 1024) : SM_BYTES;
            pl = make_plan(p, G, NT, budget, pass == 0 ? 64 : 32);
            if (pl.ok) break;
        }
    if (!pl.ok) return VL_ERR_UNSUPPORTED;

    VParams q{};
    q.nI = p->nI; q.V = p->V; q.nO = p->nO; q.nOp8 = p->nOp8; q.P = p->P; q.B = p->B; q.Bmask = p->B - 1;
    q.nB = p->nB; q.nC = p->nC; q.nGroups = p->nGroups; q.Wp = pl.Wp;
    q.ntiles = (p->nOp8 + pl.NT * 8 - 1) / (pl.NT * 8);
    q.bank_fast = p->bank_fast; q.use_th = p->use_th;
    q.vreg16 = p->d_vreg16; q.slotmeta = p->d_slotmeta; q.vinfo = p->d_vinfo; q.first_def_instr = p->d_first_def_instr;
    q.th_off = p->d_th_off; q.th = p->d_th; q.grp_off = p->d_grp_off; q.ev = p->d_ev;
    q.chunk_i0 = p->d_chunk_i0; q.chunk_i1 = p->d_chunk_i1; q.chunk_blk = p->d_chunk_blk;
    q.op_off = p->d_op_off; q.op_vreg = p->d_op_vreg; q.lo_off = p->d_lo_off; q.lo = p->d_lo;
    q.ndefs = p->d_ndefs; q.width = p->d_width; q.opflags = p->d_opflags;
    q.bank_list = p->d_bank_list;
    for (int j = 0; j < 4; ++j) q.bank_seg[j] = p->bank_seg[j];
    q.cand = d_cand; q.K = K; q.pitch = pitch; q.out = d_out; q.status = p->d_status + 1;
    q.S = pl.S; q.NS = pl.NS; q.AW = pl.AW;
    q.off_T = pl.off_T; q.off_region = pl.off_region; q.off_occ = pl.off_occ; q.off_anom = pl.off_anom;
    q.off_misc = pl.off_misc;

    const uint32_t grid = (uint32_t)((K + pl.G - 1) / pl.G);
    const bool wide = p->wmax > 31;
    cudaError_t e = cudaErrorInvalidValue;
    if (pl.NT == 256) {
        if (pl.G == 4) e = launch_w<4, 256>(wide, q, grid, pl.smem, st);
        else if (pl.G == 2) e = launch_w<2, 256>(wide, q, grid, pl.smem, st);
        else e = launch_w<1, 256>(wide, q, grid, pl.smem, st);
    } else {
        if (pl.G == 4) e = launch_w<4, 512>(wide, q, grid, pl.smem, st);
        else if (pl.G == 2) e = launch_w<2, 512>(wide, q, grid, pl.smem, st);
        else e = launch_w<1, 512>(wide, q, grid, pl.smem, st);
    }
    if (e != cudaSuccess) {
        const_cast<vl_program *>(p)->last_cuda_error = (int)e;
        return VL_ERR_CUDA;
    }
    g_vl_launches.fetch_add(1);
    return VL_OK;
}
