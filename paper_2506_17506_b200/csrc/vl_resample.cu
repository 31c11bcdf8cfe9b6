// Statistics of the re-sampling loop over verdict arrays (Section 3.4, last paragraph: the model is
// sampled again until a candidate passes or the attempts run out; Section 4: Pass@k, AvgTry, MaxTry),
// and the loop itself in batches with early exit.
//
// Work per verdict: one 16-byte record read (coalesced, once); everything else is reductions.  For
// the row counts of the re-sampling loop (hundreds to tens of thousands of rows per test case) the
// kernels are launch-latency bound; a long array is spread over several thread blocks that combine
// with 64-bit atomics (minimum and sum: the result does not depend on their order).
#include "vl_internal.cuh"

namespace {

constexpr uint32_t RS_CASES = 96;     // test cases per launch (their pointers travel as kernel arguments)
constexpr uint32_t RS_THREADS = 512;
constexpr uint32_t RS_ROWS_PER_BLOCK = RS_THREADS * 16;  // a block takes about this many rows

struct RsParams {
    const uint4 *out[RS_CASES];  // verdict arrays
    uint64_t K[RS_CASES];
    vl_sample_stats *stats;      // [cases of this launch]
    uint32_t n;
};

__global__ void k_sample_init(const RsParams q)
{
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c < q.n) { q.stats[c].first_pass = q.K[c]; q.stats[c].n_pass = 0; }
}

// grid (parts, cases): block (p, c) takes the rows p*T + t, (p + parts)*T + t, ... of case c
__global__ void __launch_bounds__(RS_THREADS) k_sample_stats(const RsParams q)
{
    const uint32_t c = blockIdx.y, tid = threadIdx.x;
    const uint64_t K = q.K[c];
    const uint64_t start = (uint64_t)blockIdx.x * RS_THREADS;
    if (start >= K) return;
    const uint4 *out = q.out[c];
    const uint64_t step = (uint64_t)gridDim.x * RS_THREADS;
    unsigned long long first = K, cnt = 0;
    for (uint64_t k = start + tid; k < K; k += step) {
        const uint4 v = __ldg(out + k);
        if (v.x & VL_PASS) {
            if (k < first) first = k;
            ++cnt;
        }
    }
#pragma unroll
    for (int d = 16; d; d >>= 1) {
        const unsigned long long f2 = __shfl_xor_sync(0xffffffffu, first, d);
        cnt += __shfl_xor_sync(0xffffffffu, cnt, d);
        first = f2 < first ? f2 : first;
    }
    __shared__ unsigned long long s_first[RS_THREADS / 32], s_cnt[RS_THREADS / 32];
    if ((tid & 31) == 0) { s_first[tid >> 5] = first; s_cnt[tid >> 5] = cnt; }
    __syncthreads();
    if (tid == 0) {
        for (uint32_t w = 1; w < RS_THREADS / 32; ++w) {
            first = s_first[w] < first ? s_first[w] : first;
            cnt += s_cnt[w];
        }
        if (cnt) {
            atomicMin(reinterpret_cast<unsigned long long *>(&q.stats[c].first_pass), first);
            atomicAdd(reinterpret_cast<unsigned long long *>(&q.stats[c].n_pass), cnt);
        }
    }
}

struct RsSumParams {
    const vl_sample_stats *stats;
    vl_resample_summary *summary;
    uint32_t n, n_k;
    uint32_t k[VL_MAX_PASS_AT];
};

// one block: the records of all test cases -> the summary
__global__ void __launch_bounds__(256) k_resample_summary(const RsSumParams q)
{
    __shared__ unsigned long long s[3 + VL_MAX_PASS_AT];  // solved, attempts summed, largest, pass@k
    const uint32_t tid = threadIdx.x;
    if (tid < 3 + VL_MAX_PASS_AT) s[tid] = 0;
    __syncthreads();
    unsigned long long solved = 0, sum = 0, mx = 0, at[VL_MAX_PASS_AT];
#pragma unroll
    for (int j = 0; j < VL_MAX_PASS_AT; ++j) at[j] = 0;
    for (uint32_t c = tid; c < q.n; c += blockDim.x) {
        if (q.stats[c].n_pass == 0) continue;
        const unsigned long long attempts = q.stats[c].first_pass + 1;
        ++solved;
        sum += attempts;
        mx = attempts > mx ? attempts : mx;
#pragma unroll
        for (int j = 0; j < VL_MAX_PASS_AT; ++j)
            if ((uint32_t)j < q.n_k && attempts <= q.k[j]) ++at[j];
    }
    if (solved) {
        atomicAdd(&s[0], solved);
        atomicAdd(&s[1], sum);
        atomicMax(&s[2], mx);
#pragma unroll
        for (int j = 0; j < VL_MAX_PASS_AT; ++j)
            if (at[j]) atomicAdd(&s[3 + j], at[j]);
    }
    __syncthreads();
    if (tid == 0) {
        vl_resample_summary r;
        r.n_cases = q.n; r.n_solved = s[0]; r.sum_tries = s[1]; r.max_tries = s[2];
        for (int j = 0; j < VL_MAX_PASS_AT; ++j) r.pass_at[j] = s[3 + j];
        *q.summary = r;
    }
}

// records of cases [c0, c0 + m) into d_stats + c0
cudaError_t launch_stats(uint32_t m, const vl_verdict *const *d_out, const uint64_t *K, vl_sample_stats *d_stats,
                         cudaStream_t st, uint32_t max_parts)
{
    RsParams q;
    uint64_t kmax = 0;
    for (uint32_t j = 0; j < m; ++j) {
        q.out[j] = reinterpret_cast<const uint4 *>(d_out[j]);
        q.K[j] = K[j];
        kmax = K[j] > kmax ? K[j] : kmax;
    }
    q.stats = d_stats;
    q.n = m;
    k_sample_init<<<1, RS_CASES, 0, st>>>(q);
    g_vl_launches.fetch_add(1);
    if (kmax) {
        uint64_t parts = (kmax + RS_ROWS_PER_BLOCK - 1) / RS_ROWS_PER_BLOCK;
        if (parts > max_parts) parts = max_parts;
        k_sample_stats<<<dim3((uint32_t)parts, m), RS_THREADS, 0, st>>>(q);
        g_vl_launches.fetch_add(1);
    }
    return cudaGetLastError();
}

}  // namespace

extern "C" int vl_resample_stats(int device, uint32_t n, const vl_verdict *const *d_out, const uint64_t *K,
                                 uint32_t n_k, const uint32_t *k, vl_sample_stats *d_stats,
                                 vl_resample_summary *d_summary, void *stream)
{
    if (n_k > VL_MAX_PASS_AT || (n_k && !k)) return VL_ERR_INVALID_ARG;
    if (n && (!d_out || !K || !d_stats)) return VL_ERR_INVALID_ARG;
    if (((uintptr_t)d_stats & 7) || ((uintptr_t)d_summary & 7)) return VL_ERR_INVALID_ARG;
    for (uint32_t j = 0; j < n; ++j)
        if (K[j] && (!d_out[j] || ((uintptr_t)d_out[j] & 15))) return VL_ERR_INVALID_ARG;
    if (n == 0 && !d_summary) return VL_OK;
    if (cudaSetDevice(device) != cudaSuccess) return VL_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    for (uint32_t c0 = 0; c0 < n; c0 += RS_CASES) {
        const uint32_t m = n - c0 < RS_CASES ? n - c0 : RS_CASES;
        // at most 4 thread blocks per multiprocessor work on one verdict array
        if (launch_stats(m, d_out + c0, K + c0, d_stats + c0, st, 4u * (uint32_t)vl_device_sm_count(device)) != cudaSuccess)
            return VL_ERR_CUDA;
    }
    if (d_summary) {
        RsSumParams s;
        s.stats = d_stats; s.summary = d_summary; s.n = n; s.n_k = n_k;
        for (uint32_t j = 0; j < VL_MAX_PASS_AT; ++j) s.k[j] = j < n_k ? k[j] : 0;
        k_resample_summary<<<1, 256, 0, st>>>(s);
        g_vl_launches.fetch_add(1);
        if (cudaGetLastError() != cudaSuccess) return VL_ERR_CUDA;
    }
    return VL_OK;
}

extern "C" int vl_verify_until_pass(vl_program *p, const uint16_t *d_cand, uint64_t K, uint64_t pitch,
                                    uint64_t batch_rows, vl_verdict *d_out, uint64_t *rows_checked,
                                    uint64_t *first_pass, void *stream)
{
    if (!p || !rows_checked || !first_pass || batch_rows == 0) return VL_ERR_INVALID_ARG;
    *rows_checked = 0;
    *first_pass = K;
    if (!p->live_ok) return VL_ERR_LIVENESS_NOT_RUN;
    if (K == 0) return VL_OK;
    if (!d_cand || !d_out || ((uintptr_t)d_out & 15)) return VL_ERR_INVALID_ARG;
    VL_CUDA(p, cudaSetDevice(p->device));
    if (!p->d_rs) VL_CUDA(p, cudaMalloc(&p->d_rs, sizeof(vl_sample_stats)));
    if (!p->h_rs) VL_CUDA(p, cudaMallocHost(&p->h_rs, sizeof(vl_sample_stats)));
    cudaStream_t st = (cudaStream_t)stream;
    for (uint64_t b0 = 0; b0 < K; b0 += batch_rows) {
        const uint64_t nb = K - b0 < batch_rows ? K - b0 : batch_rows;
        const int rc = vl_verify(p, d_cand + b0 * pitch, nb, pitch, d_out + b0, stream);
        if (rc != VL_OK) return rc;
        const vl_verdict *outs = d_out + b0;
        VL_CUDA(p, launch_stats(1, &outs, &nb, p->d_rs, st, 4u * (uint32_t)vl_sm_count(p)));
        VL_CUDA(p, cudaMemcpyAsync(p->h_rs, p->d_rs, sizeof(vl_sample_stats), cudaMemcpyDeviceToHost, st));
        VL_CUDA(p, cudaStreamSynchronize(st));
        *rows_checked = b0 + nb;
        if (p->h_rs->n_pass) {
            *first_pass = b0 + p->h_rs->first_pass;
            break;
        }
    }
    return VL_OK;
}
