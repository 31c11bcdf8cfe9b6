// Block-level liveness for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need an answer: a
// serving process that reserved all of HBM for its own pools at start-up, a plugin running under a
// memory budget it does not own, or a latency-critical loop where the device-wide synchronisation
// that an allocation implies is not acceptable.  vl_liveness allocates its working sets; this entry
// point does not.  The per-block read/write bitsets it needs live in one file-scope device array of
// fixed size, so a program is accepted only if those sets fit, and every call on a device shares
// that one array.
#include <mutex>

#include "vl_internal.cuh"

#define NA_THREADS 128
// Fixed scratch: VL_STATIC_SCRATCH_WORDS 32-bit words (1 MiB) plus a small header, per GPU that loads
// the library, held until exit.
#define NA_SCRATCH_WORDS (VL_STATIC_SCRATCH_WORDS + 16u)
#define NA_HEADER_WORDS 16u  // words 0, 1: status bits of the last call (cleared by the call itself)
#define ST_BAD_INDEX 32u     // an operand names no vreg of the program, or a successor no block

static __device__ __align__(256) uint32_t g_na_scratch[NA_SCRATCH_WORDS];

namespace {
std::mutex g_na_mutex;
uint32_t *g_na_ptr[64] = {nullptr};  // device address of g_na_scratch, per device ordinal
}  // namespace

// One block of threads per basic block: read-before-write set and write set of the block, built in
// shared memory by a sequential walk (reads of an instruction come before its writes), then stored
// to the scratch rows of this basic block.  Every word of both rows is written, so nothing of an
// earlier call survives.
__global__ void k_na_block_sets(const uint32_t *__restrict__ blk_off, const uint32_t *__restrict__ op_off,
                                const uint8_t *__restrict__ ndefs, const uint32_t *__restrict__ op_vreg, uint32_t Wv,
                                uint32_t n_vregs, uint32_t *blk_use, uint32_t *blk_def, uint32_t *status)
{
    extern __shared__ uint32_t sm[];
    uint32_t *s_use = sm, *s_def = sm + Wv;
    const uint32_t b = blockIdx.x;

    for (uint32_t w = threadIdx.x; w < 2 * Wv; w += NA_THREADS) sm[w] = 0;
    __syncthreads();
    if (threadIdx.x == 0) {
        bool bad = false;
        for (uint32_t i = blk_off[b]; i < blk_off[b + 1]; ++i) {
            const uint32_t o0 = op_off[i], o1 = op_off[i + 1], nd = ndefs[i];
            // (the program is not validated on the host: an id outside the program is skipped and reported)
            for (uint32_t o = o0 + nd; o < o1; ++o) {
                const uint32_t v = op_vreg[o];
                if (v >= n_vregs) { bad = true; continue; }
                if (!((s_def[v >> 5] >> (v & 31)) & 1u)) s_use[v >> 5] |= 1u << (v & 31);
            }
            for (uint32_t o = o0; o < o0 + nd && o < o1; ++o) {
                const uint32_t v = op_vreg[o];
                if (v >= n_vregs) { bad = true; continue; }
                s_def[v >> 5] |= 1u << (v & 31);
            }
        }
        if (bad) atomicOr(status + 1, ST_BAD_INDEX);
    }
    __syncthreads();
    for (uint32_t w = threadIdx.x; w < Wv; w += NA_THREADS) {
        blk_use[(size_t)b * Wv + w] = s_use[w];
        blk_def[(size_t)b * Wv + w] = s_def[w];
    }
}

// Backward dataflow to the least fixed point, one thread per bitset word (words do not interact).
// The caller's live_in / live_out are cleared here before iterating.
__global__ void k_na_fixed_point(uint32_t nB, uint32_t Wv, const uint32_t *__restrict__ succ_off,
                                 const uint32_t *__restrict__ succ, const uint32_t *__restrict__ blk_use,
                                 const uint32_t *__restrict__ blk_def, uint32_t *live_in, uint32_t *live_out,
                                 uint32_t *status)
{
    const uint32_t w = blockIdx.x * NA_THREADS + threadIdx.x;
    if (w >= Wv) return;
    for (uint32_t b = 0; b < nB; ++b) {
        live_in[(size_t)b * Wv + w] = 0;
        live_out[(size_t)b * Wv + w] = 0;
    }
    bool changed = true, bad = false;
    for (uint32_t sweep = 0; sweep < nB + 2 && changed; ++sweep) {
        changed = false;
        for (uint32_t n = 0; n < nB; ++n) {
            const uint32_t b = nB - 1 - n;
            uint32_t o = 0;
            for (uint32_t e = succ_off[b]; e < succ_off[b + 1]; ++e) {
                const uint32_t sb = succ ? succ[e] : nB;
                if (sb >= nB) { bad = true; continue; }  // not a block of the program: skipped and reported
                o |= live_in[(size_t)sb * Wv + w];
            }
            const uint32_t in = blk_use[(size_t)b * Wv + w] | (o & ~blk_def[(size_t)b * Wv + w]);
            if (o != live_out[(size_t)b * Wv + w] || in != live_in[(size_t)b * Wv + w]) changed = true;
            live_out[(size_t)b * Wv + w] = o;
            live_in[(size_t)b * Wv + w] = in;
        }
    }
    if (changed) atomicOr(status, ST_NO_CONVERGE);
    if (bad) atomicOr(status + 1, ST_BAD_INDEX);
}

extern "C" int vl_block_liveness_static(int device, uint32_t n_blocks, uint32_t n_vregs,
                                        const uint32_t *d_block_instr_off, const uint32_t *d_succ_off,
                                        const uint32_t *d_succ, const uint32_t *d_instr_op_off,
                                        const uint8_t *d_instr_n_defs, const uint32_t *d_op_vreg,
                                        uint32_t *d_live_in, uint32_t *d_live_out, void *cuda_stream)
{
    if (device < 0 || device >= 64 || n_blocks == 0) return VL_ERR_INVALID_ARG;
    if (!d_block_instr_off || !d_succ_off || !d_instr_op_off || !d_instr_n_defs || !d_op_vreg || !d_live_in || !d_live_out)
        return VL_ERR_INVALID_ARG;
    if (n_vregs > 65535) return VL_ERR_UNSUPPORTED;
    const uint32_t Wv = n_vregs ? (n_vregs + 31) / 32 : 1;
    // two bitset rows per basic block must fit the fixed array
    if (2ull * n_blocks * Wv > (uint64_t)(NA_SCRATCH_WORDS - NA_HEADER_WORDS)) return VL_ERR_UNSUPPORTED;
    if (cudaSetDevice(device) != cudaSuccess) return VL_ERR_CUDA;

    uint32_t *scratch;
    {   // once per device, with that device current: the device address behind the symbol
        std::lock_guard<std::mutex> lock(g_na_mutex);
        if (!g_na_ptr[device]) {
            void *ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_na_scratch) != cudaSuccess || !ptr) return VL_ERR_CUDA;
            g_na_ptr[device] = static_cast<uint32_t *>(ptr);
        }
        scratch = g_na_ptr[device];
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    uint32_t *status = scratch;
    uint32_t *blk_use = scratch + NA_HEADER_WORDS;
    uint32_t *blk_def = blk_use + (size_t)n_blocks * Wv;

    if (cudaMemsetAsync(status, 0, 2 * sizeof(uint32_t), st) != cudaSuccess) return VL_ERR_CUDA;
    k_na_block_sets<<<n_blocks, NA_THREADS, 2 * Wv * sizeof(uint32_t), st>>>(d_block_instr_off, d_instr_op_off,
                                                                             d_instr_n_defs, d_op_vreg, Wv, n_vregs, blk_use,
                                                                             blk_def, status);
    k_na_fixed_point<<<(Wv + NA_THREADS - 1) / NA_THREADS, NA_THREADS, 0, st>>>(n_blocks, Wv, d_succ_off, d_succ, blk_use,
                                                                               blk_def, d_live_in, d_live_out, status);
    g_vl_launches.fetch_add(2);
    if (cudaGetLastError() != cudaSuccess) return VL_ERR_CUDA;
    uint32_t h_status[2] = {0, 0};
    if (cudaMemcpyAsync(h_status, status, 2 * sizeof(uint32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess) return VL_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return VL_ERR_CUDA;
    if (h_status[1] & ST_BAD_INDEX) return VL_ERR_MALFORMED_PROGRAM;
    return (h_status[0] & ST_NO_CONVERGE) ? VL_ERR_NO_CONVERGE : VL_OK;
}
