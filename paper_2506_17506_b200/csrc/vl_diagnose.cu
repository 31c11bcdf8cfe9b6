// Diagnostics of one candidate, for feedback to the sampler, and the registers occupied at every
// definition point, for decoding that masks them out (Section 4.5, last paragraph).
// Diagnostics (Section 4.5 sorts failures into
// dataflow violations and hardware-constraint violations; Section 6 proposes the verifier's findings
// as a training signal): every (instruction, defined vreg, other vreg) overlap, the violation kinds
// raised at every instruction, and the extra read cycles per register bank.
//
// This is not the hot path: one row, one warp per instruction, the per-instruction live-after
// lists of vl_liveness read as they are.  The numbers agree with the verdict of vl_verify for the
// same row: the overlap count is conflict_pairs, the histogram sums to bank_conflicts, the lowest
// instruction with a kind is first_violation_instr.
#include "vl_internal.cuh"

namespace {

struct DParams {
    uint32_t nI, nO, V, P, B;
    const uint32_t *op_off, *op_vreg, *lo_off, *lo;
    const uint8_t *ndefs, *width;
    const uint4 *vcons;
    const uint16_t *rs_prefix;
    const uint16_t *row;
    unsigned long long *T64;  // [V] (first occurrence << 16) | value there
    uint64_t cap;
    vl_conflict *conflicts;
    unsigned long long *n_conflicts;
    uint8_t *kinds;
    unsigned long long *bank_hist;
};

__global__ void k_diag_init(const DParams q)
{
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t < q.V) q.T64[t] = ~0ull;
    if (t == 0) *q.n_conflicts = 0;
    if (q.bank_hist && t < q.B) q.bank_hist[t] = 0;
}

// first occurrence wins: the smallest (operand index, value) pair per vreg
__global__ void k_diag_table(const DParams q)
{
    const uint32_t o = blockIdx.x * blockDim.x + threadIdx.x;
    if (o < q.nO) atomicMin(&q.T64[q.op_vreg[o]], ((unsigned long long)o << 16) | q.row[o]);
}

__device__ __forceinline__ bool overlap(uint32_t a, uint32_t wa, uint32_t b, uint32_t wb)
{
    return a < b + wb && b < a + wa;
}

// one warp per instruction: the lanes share out the operands and the live-after list
constexpr uint32_t DIAG_WARPS = 4;
__global__ void __launch_bounds__(DIAG_WARPS * 32) k_diag_instr(const DParams q)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t i = blockIdx.x * DIAG_WARPS + (threadIdx.x >> 5);
    if (i >= q.nI) return;
    const uint32_t o0 = q.op_off[i], o1 = q.op_off[i + 1], nd = q.ndefs[i];
    const uint32_t l0 = q.lo_off[i], l1 = q.lo_off[i + 1];
    auto T = [&](uint32_t v) { return (uint32_t)(q.T64[v] & 0xFFFFu); };
    auto emit = [&](uint32_t v, uint32_t u) {
        const unsigned long long k = atomicAdd(q.n_conflicts, 1ull);
        if (k < q.cap) q.conflicts[k] = vl_conflict{i, v, u};
    };
    uint32_t kinds = 0;
    for (uint32_t o = o0 + lane; o < o1; o += 32)
        if (q.row[o] != T(q.op_vreg[o])) kinds |= VL_INCONSISTENT;
    for (uint32_t d = o0; d < o0 + nd; ++d) {
        const uint32_t v = q.op_vreg[d], s = T(v), w = q.width[v];
        if (lane == 0) {
            bool unreal = s + w > q.P;
            if (q.vcons) {
                const uint4 vc = q.vcons[v];
                const uint32_t clo = vc.x & 0xFFFFu, chi = vc.x >> 16, al = vc.y;
                unreal = unreal || (al > 1 && s != __umulhi(s, vc.z) * al) || s < clo || s + w > chi;
                if (q.rs_prefix) unreal = unreal || q.rs_prefix[min(s + w, q.P)] != q.rs_prefix[min(s, q.P)];
            }
            if (unreal) kinds |= VL_OUT_OF_RANGE;
        }
        for (uint32_t e = l0 + lane; e < l1; e += 32) {  // vregs live after the instruction
            const uint32_t u = q.lo[e];
            if (u != v && overlap(s, w, T(u), q.width[u])) { emit(v, u); kinds |= VL_INTERFERENCE; }
        }
        for (uint32_t d2 = o0 + lane; d2 < o0 + nd; d2 += 32) {  // vregs it also defines that are dead afterwards
            const uint32_t u = q.op_vreg[d2];
            if (u == v) continue;
            uint32_t a = l0, b = l1;  // the list is ascending
            while (a < b) {
                const uint32_t m = (a + b) >> 1;
                if (q.lo[m] < u) a = m + 1; else b = m;
            }
            if (a < l1 && q.lo[a] == u) continue;
            if (overlap(s, w, T(u), q.width[u])) { emit(v, u); kinds |= VL_INTERFERENCE; }
        }
    }
    kinds = __reduce_or_sync(0xffffffffu, kinds);
    if (q.kinds && lane == 0) q.kinds[i] = (uint8_t)kinds;
    if (q.bank_hist) {
        // a read costs a cycle if an earlier read of this instruction uses another register of its bank
        // and no earlier read uses the same register
        for (uint32_t a = o0 + nd + lane; a < o1; a += 32) {
            const uint32_t ta = T(q.op_vreg[a]);
            bool dup = false, shared = false;
            for (uint32_t b = o0 + nd; b < a; ++b) {
                const uint32_t tb = T(q.op_vreg[b]);
                dup = dup || tb == ta;
                shared = shared || tb % q.B == ta % q.B;
            }
            if (!dup && shared) atomicAdd(&q.bank_hist[ta % q.B], 1ull);
        }
    }
}

// Occupied registers per instruction: one warp per instruction ORs the ranges of the vregs live
// after it (own definitions left out, reserved registers added) into a mask in shared memory and
// writes the mask out.  W = words per mask.
constexpr uint32_t OCC_WARPS = 4;
__global__ void __launch_bounds__(OCC_WARPS * 32) k_occupied(const DParams q, uint32_t W, uint32_t *masks)
{
    extern __shared__ uint32_t s_mask[];
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t i = blockIdx.x * OCC_WARPS + warp;
    if (i >= q.nI) return;
    uint32_t *m = s_mask + warp * W;
    for (uint32_t j = lane; j < W; j += 32) {  // reserved registers: bit r set iff the prefix count steps at r
        uint32_t x = 0;
        if (q.rs_prefix)
            for (uint32_t b = 0; b < 32 && j * 32 + b < q.P; ++b)
                x |= (uint32_t)(q.rs_prefix[j * 32 + b + 1] != q.rs_prefix[j * 32 + b]) << b;
        m[j] = x;
    }
    __syncwarp();
    const uint32_t o0 = q.op_off[i], nd = q.ndefs[i];
    for (uint32_t e = q.lo_off[i] + lane; e < q.lo_off[i + 1]; e += 32) {
        const uint32_t u = q.lo[e];
        bool own = false;
        for (uint32_t d = o0; d < o0 + nd; ++d) own = own || q.op_vreg[d] == u;
        if (own) continue;
        const uint32_t t = (uint32_t)(q.T64[u] & 0xFFFFu);
        const uint32_t end = min(t + q.width[u], q.P);
        for (uint32_t r = t; r < end;) {  // word by word
            const uint32_t hi = min(end, (r | 31u) + 1u), n = hi - r;
            atomicOr(&m[r >> 5], (n == 32 ? 0xFFFFFFFFu : ((1u << n) - 1u)) << (r & 31));
            r = hi;
        }
    }
    __syncwarp();
    for (uint32_t j = lane; j < W; j += 32) masks[(size_t)i * W + j] = m[j];
}

}  // namespace

extern "C" int vl_occupied_masks(vl_program *p, const uint16_t *d_row, uint32_t *d_masks, void *stream)
{
    if (!p || !d_row || !d_masks) return VL_ERR_INVALID_ARG;
    if (((uintptr_t)d_row & 1) || ((uintptr_t)d_masks & 3)) return VL_ERR_INVALID_ARG;
    if (p->live_pending) {
        const int rc = vl_live_settle(p);
        if (rc != VL_OK) return rc;
    }
    if (!p->live_ok) return VL_ERR_LIVENESS_NOT_RUN;
    VL_CUDA(p, cudaSetDevice(p->device));
    if (!p->d_diag_T) VL_CUDA(p, cudaMalloc(&p->d_diag_T, sizeof(unsigned long long) * (p->V ? p->V : 1)));
    if (!p->d_diag_n) VL_CUDA(p, cudaMalloc(&p->d_diag_n, sizeof(unsigned long long)));
    cudaStream_t st = (cudaStream_t)stream;
    DParams q{};
    q.nI = p->nI; q.nO = p->nO; q.V = p->V; q.P = p->P; q.B = p->B;
    q.op_off = p->d_op_off; q.op_vreg = p->d_op_vreg; q.lo_off = p->d_lo_off; q.lo = p->d_lo;
    q.ndefs = p->d_ndefs; q.width = p->d_width; q.rs_prefix = p->d_rs_prefix;
    q.row = d_row; q.T64 = p->d_diag_T; q.n_conflicts = p->d_diag_n;
    const uint32_t W = (p->P + 31) / 32;
    k_diag_init<<<(p->V + 255) / 256 + 1, 256, 0, st>>>(q);
    if (p->nO) k_diag_table<<<(p->nO + 255) / 256, 256, 0, st>>>(q);
    if (p->nI) k_occupied<<<(p->nI + OCC_WARPS - 1) / OCC_WARPS, OCC_WARPS * 32, OCC_WARPS * W * sizeof(uint32_t), st>>>(q, W, d_masks);
    g_vl_launches.fetch_add(1 + (p->nO ? 1 : 0) + (p->nI ? 1 : 0));
    VL_CUDA(p, cudaGetLastError());
    return VL_OK;
}

extern "C" int vl_diagnose(vl_program *p, const uint16_t *d_row, uint64_t cap, vl_conflict *d_conflicts,
                           uint64_t *d_n_conflicts, uint8_t *d_kinds, uint64_t *d_bank_hist, void *stream)
{
    if (!p || !d_row || !d_n_conflicts || (cap && !d_conflicts)) return VL_ERR_INVALID_ARG;
    if (((uintptr_t)d_row & 1) || ((uintptr_t)d_conflicts & 3) || ((uintptr_t)d_n_conflicts & 7) ||
        ((uintptr_t)d_bank_hist & 7))
        return VL_ERR_INVALID_ARG;
    if (p->live_pending) {
        const int rc = vl_live_settle(p);
        if (rc != VL_OK) return rc;
    }
    if (!p->live_ok) return VL_ERR_LIVENESS_NOT_RUN;
    VL_CUDA(p, cudaSetDevice(p->device));
    if (!p->d_diag_T) VL_CUDA(p, cudaMalloc(&p->d_diag_T, sizeof(unsigned long long) * (p->V ? p->V : 1)));
    cudaStream_t st = (cudaStream_t)stream;
    DParams q{};
    q.nI = p->nI; q.nO = p->nO; q.V = p->V; q.P = p->P; q.B = p->B;
    q.op_off = p->d_op_off; q.op_vreg = p->d_op_vreg; q.lo_off = p->d_lo_off; q.lo = p->d_lo;
    q.ndefs = p->d_ndefs; q.width = p->d_width; q.vcons = p->d_vcons; q.rs_prefix = p->d_rs_prefix;
    q.row = d_row; q.T64 = p->d_diag_T; q.cap = cap; q.conflicts = d_conflicts;
    q.n_conflicts = reinterpret_cast<unsigned long long *>(d_n_conflicts);
    q.kinds = d_kinds; q.bank_hist = reinterpret_cast<unsigned long long *>(d_bank_hist);
    const uint32_t n0 = p->V > p->B ? p->V : p->B;
    k_diag_init<<<(n0 + 255) / 256 + 1, 256, 0, st>>>(q);
    if (p->nO) k_diag_table<<<(p->nO + 255) / 256, 256, 0, st>>>(q);
    if (p->nI) k_diag_instr<<<(p->nI + DIAG_WARPS - 1) / DIAG_WARPS, DIAG_WARPS * 32, 0, st>>>(q);
    g_vl_launches.fetch_add(1 + (p->nO ? 1 : 0) + (p->nI ? 1 : 0));
    VL_CUDA(p, cudaGetLastError());
    return VL_OK;
}
