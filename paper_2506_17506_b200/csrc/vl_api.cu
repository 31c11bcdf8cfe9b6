// C ABI entry points: program handle, validation, host-buffer verify, error strings.
#include <algorithm>
#include <cstring>
#include <mutex>
#include <new>

#include "vl_internal.cuh"

std::atomic<uint64_t> g_vl_launches{0};

// Lane streams are per device and shared by every handle on it; they live until the process exits.
#define VL_MAX_DEVICES 64
static std::mutex g_lane_mutex;
static cudaStream_t g_lanes[VL_MAX_DEVICES][VL_STREAMS];  // the lanes, two side streams of a liveness run, the liveness stream
static bool g_lanes_made[VL_MAX_DEVICES];

int vl_lane_streams(vl_program *p, cudaStream_t **lanes)
{
    if (p->device < 0 || p->device >= VL_MAX_DEVICES) return VL_ERR_UNSUPPORTED;
    {
        std::lock_guard<std::mutex> lock(g_lane_mutex);
        if (!g_lanes_made[p->device]) {
            for (int l = 0; l < VL_LANES + 2; ++l)
                VL_CUDA(p, cudaStreamCreateWithFlags(&g_lanes[p->device][l], cudaStreamNonBlocking));
            // the liveness stream: its small kernels go first wherever a multiprocessor has room
            int least = 0, greatest = 0;
            VL_CUDA(p, cudaDeviceGetStreamPriorityRange(&least, &greatest));
            VL_CUDA(p, cudaStreamCreateWithPriority(&g_lanes[p->device][VL_LIVE_STREAM], cudaStreamNonBlocking, greatest));
            g_lanes_made[p->device] = true;
        }
    }
    if (!p->ev_fork) VL_CUDA(p, cudaEventCreateWithFlags(&p->ev_fork, cudaEventDisableTiming));
    if (!p->ev_pre) VL_CUDA(p, cudaEventCreateWithFlags(&p->ev_pre, cudaEventDisableTiming));
    for (int l = 0; l < 3; ++l)
        if (!p->ev_side[l]) VL_CUDA(p, cudaEventCreateWithFlags(&p->ev_side[l], cudaEventDisableTiming));
    for (int l = 0; l < VL_LANES; ++l)
        if (!p->ev_join[l]) VL_CUDA(p, cudaEventCreateWithFlags(&p->ev_join[l], cudaEventDisableTiming));
    *lanes = g_lanes[p->device];
    return VL_OK;
}

static int validate(const vl_program_desc *d)
{
    if (!d) return VL_ERR_INVALID_ARG;
    if (!d->block_instr_off || !d->succ_off || !d->instr_op_off) return VL_ERR_INVALID_ARG;
    if (d->n_edges && !d->succ) return VL_ERR_INVALID_ARG;
    if (d->n_instrs && !d->instr_n_defs) return VL_ERR_INVALID_ARG;
    if (d->n_operands && !d->op_vreg) return VL_ERR_INVALID_ARG;
    if (d->n_vregs && !d->vreg_width) return VL_ERR_INVALID_ARG;
    if (d->n_blocks == 0 || d->P == 0 || d->P > 65535 || d->B == 0) return VL_ERR_INVALID_ARG;
    if (d->n_vregs > 65535) return VL_ERR_UNSUPPORTED;
    if (d->n_operands > 0xFFFFFFF0u - 64 || d->n_instrs > 0x7FFFFFF0u) return VL_ERR_UNSUPPORTED;

    if (d->block_instr_off[0] != 0 || d->block_instr_off[d->n_blocks] != d->n_instrs) return VL_ERR_MALFORMED_PROGRAM;
    for (uint32_t b = 0; b < d->n_blocks; ++b)
        if (d->block_instr_off[b] > d->block_instr_off[b + 1]) return VL_ERR_MALFORMED_PROGRAM;
    if (d->succ_off[0] != 0 || d->succ_off[d->n_blocks] != d->n_edges) return VL_ERR_MALFORMED_PROGRAM;
    for (uint32_t b = 0; b < d->n_blocks; ++b)
        if (d->succ_off[b] > d->succ_off[b + 1]) return VL_ERR_MALFORMED_PROGRAM;
    for (uint32_t e = 0; e < d->n_edges; ++e)
        if (d->succ[e] >= d->n_blocks) return VL_ERR_MALFORMED_PROGRAM;
    if (d->instr_op_off[0] != 0 || d->instr_op_off[d->n_instrs] != d->n_operands) return VL_ERR_MALFORMED_PROGRAM;
    for (uint32_t i = 0; i < d->n_instrs; ++i) {
        uint32_t o0 = d->instr_op_off[i], o1 = d->instr_op_off[i + 1];
        if (o0 > o1 || o1 > d->n_operands) return VL_ERR_MALFORMED_PROGRAM;
        if (d->instr_n_defs[i] > o1 - o0) return VL_ERR_MALFORMED_PROGRAM;
    }
    for (uint32_t o = 0; o < d->n_operands; ++o)
        if (d->op_vreg[o] >= d->n_vregs) return VL_ERR_MALFORMED_PROGRAM;
    for (uint32_t v = 0; v < d->n_vregs; ++v)
        if (d->vreg_width[v] == 0) return VL_ERR_MALFORMED_PROGRAM;
    for (uint32_t i = 0; i < d->n_instrs; ++i) {  // one instruction must not define a vreg twice
        uint32_t o0 = d->instr_op_off[i], nd = d->instr_n_defs[i];
        for (uint32_t a = 0; a < nd; ++a)
            for (uint32_t b = a + 1; b < nd; ++b)
                if (d->op_vreg[o0 + a] == d->op_vreg[o0 + b]) return VL_ERR_MALFORMED_PROGRAM;
    }
    return VL_OK;
}

template <typename T>
static cudaError_t upload(T **dst, const T *src, size_t n)
{
    cudaError_t e = cudaMalloc((void **)dst, std::max<size_t>(n, 1) * sizeof(T) + 64);
    if (e != cudaSuccess) return e;
    if (n) e = cudaMemcpy(*dst, src, n * sizeof(T), cudaMemcpyHostToDevice);
    return e;
}

extern "C" int vl_program_create(const vl_program_desc *d, int device, vl_program **out)
{
    if (!out) return VL_ERR_INVALID_ARG;
    int rc = validate(d);
    if (rc != VL_OK) return rc;
    vl_program *p = new (std::nothrow) vl_program();
    if (!p) return VL_ERR_CUDA;
    p->device = device;
    p->nB = d->n_blocks; p->nI = d->n_instrs; p->V = d->n_vregs; p->nO = d->n_operands; p->nE = d->n_edges;
    p->P = d->P; p->B = d->B;
    p->Wv = std::max(1u, (p->V + 31) / 32);
    p->nOp8 = std::max(8u, (p->nO + 7) / 8 * 8);
    p->nOpT = (p->nOp8 + 4095u) / 4096u * 4096u + 4096u;  // (the table kernel reads its metadata up to two tiles ahead)
    p->wmax = 1;
    for (uint32_t v = 0; v < p->V; ++v) p->wmax = std::max<uint32_t>(p->wmax, d->vreg_width[v]);
    p->h_blk_off.assign(d->block_instr_off, d->block_instr_off + p->nB + 1);
    p->h_op_off.assign(d->instr_op_off, d->instr_op_off + p->nI + 1);

    cudaError_t e = cudaSetDevice(device);
    if (e == cudaSuccess) e = upload(&p->d_blk_off, d->block_instr_off, (size_t)p->nB + 1);
    if (e == cudaSuccess) e = upload(&p->d_succ_off, d->succ_off, (size_t)p->nB + 1);
    if (e == cudaSuccess) e = upload(&p->d_succ, d->succ, (size_t)p->nE);
    if (e == cudaSuccess) e = upload(&p->d_op_off, d->instr_op_off, (size_t)p->nI + 1);
    if (e == cudaSuccess) e = upload(&p->d_ndefs, d->instr_n_defs, (size_t)p->nI);
    if (e == cudaSuccess) e = upload(&p->d_op_vreg, d->op_vreg, (size_t)p->nO);
    if (e == cudaSuccess) e = upload(&p->d_width, d->vreg_width, (size_t)p->V);
    {   // instructions grouped by their number of distinct sources (2, 3, 4), for the bank tally
        std::vector<uint2> cls[3];
        for (uint32_t i = 0; i < p->nI; ++i) {
            uint32_t ids[4], n = 0;
            bool many = false;
            for (uint32_t o = d->instr_op_off[i] + d->instr_n_defs[i]; o < d->instr_op_off[i + 1]; ++o) {
                const uint32_t v = d->op_vreg[o];
                bool dup = false;
                for (uint32_t k = 0; k < n; ++k) dup |= (ids[k] == v);
                if (dup) continue;
                if (n == 4) { many = true; break; }
                ids[n++] = v;
            }
            if (many) { p->bank_many = 1; continue; }
            if (n < 2) continue;
            for (uint32_t k = n; k < 4; ++k) ids[k] = ids[0];  // unused slots repeat the first source
            cls[n - 2].push_back(make_uint2(ids[0] | (ids[1] << 16), ids[2] | (ids[3] << 16)));
        }
        std::vector<uint2> all;
        p->bank_seg[0] = 0;
        for (int c = 0; c < 3; ++c) {
            all.insert(all.end(), cls[c].begin(), cls[c].end());
            p->bank_seg[c + 1] = (uint32_t)all.size();
        }
        if (e == cudaSuccess) e = upload(&p->d_bank_list, all.data(), all.size());
    }
    {   // The dictionary form of a candidate row (Section 3.1: one vreg -> register dictionary per basic
        // block): one entry per (block, vreg occurring in the block), blocks in order, a block's vregs
        // in order of first occurrence.  The operand tables of the table kernels, for rows in that
        // form: vreg of every entry, first-entry bits (the entry of the lowest block that uses the
        // vreg gives the table value), and the instruction a differing entry is reported at.
        std::vector<uint32_t> dict_instr;
        std::vector<uint32_t> stamp(p->V ? p->V : 1, 0xFFFFFFFFu);
        std::vector<uint8_t> has_entry(p->V ? p->V : 1, 0);
        std::vector<uint8_t> is_first;
        p->h_dict_off.assign(1, 0u);
        for (uint32_t b = 0; b < p->nB; ++b) {
            for (uint32_t i = d->block_instr_off[b]; i < d->block_instr_off[b + 1]; ++i)
                for (uint32_t o = d->instr_op_off[i]; o < d->instr_op_off[i + 1]; ++o) {
                    const uint32_t v = d->op_vreg[o];
                    if (stamp[v] == b) continue;
                    stamp[v] = b;
                    p->h_dict_vreg.push_back(v);
                    dict_instr.push_back(i);
                    is_first.push_back(has_entry[v] ? 0 : 1);
                    has_entry[v] = 1;
                }
            p->h_dict_off.push_back((uint32_t)p->h_dict_vreg.size());
        }
        p->nD = (uint32_t)p->h_dict_vreg.size();
        p->nD8 = std::max(8u, (p->nD + 7) / 8 * 8);
        p->nDT = (p->nD8 + 4095u) / 4096u * 4096u + 4096u;
        std::vector<uint16_t> v16((size_t)p->nD8 + 8, (uint16_t)p->V);
        std::vector<uint64_t> slot((size_t)p->nD8 / 8, 0);
        std::vector<uint4> off((size_t)p->nDT / 4, make_uint4(p->V * 16u, p->V * 16u, p->V * 16u, p->V * 16u));
        std::vector<uint8_t> f4((size_t)p->nDT / 4, 0);
        dict_instr.resize(p->nD8, 0);
        for (uint32_t e2 = 0; e2 < p->nD8; ++e2) {
            if (e2 < p->nD) {
                const uint32_t v = p->h_dict_vreg[e2];
                v16[e2] = (uint16_t)v;
                uint32_t *w = &off[e2 / 4].x;
                w[e2 % 4] = v * 16u;
                if (is_first[e2]) { slot[e2 / 8] |= 1ull << (e2 % 8); f4[e2 / 4] |= (uint8_t)(1u << (e2 % 4)); }
            } else {
                slot[e2 / 8] |= 1ull << (e2 % 8);  // padding column: writes the spare table entry, never compared
            }
        }
        if (e == cudaSuccess) e = upload(&p->d_dict_vreg16, v16.data(), v16.size());
        if (e == cudaSuccess) e = upload(&p->d_dict_slotmeta, slot.data(), slot.size());
        if (e == cudaSuccess) e = upload(&p->d_dict_opoff, off.data(), off.size());
        if (e == cudaSuccess) e = upload(&p->d_dict_first4, f4.data(), f4.size());
        if (e == cudaSuccess) e = upload(&p->d_dict_instr, dict_instr.data(), dict_instr.size());
    }
    if (e == cudaSuccess) e = cudaMalloc((void **)&p->d_status, 64);
    if (e == cudaSuccess) e = cudaMemset(p->d_status, 0, 64);
    if (e != cudaSuccess) {
        p->last_cuda_error = (int)e;
        vl_program_destroy(p);
        return VL_ERR_CUDA;
    }
    *out = p;
    return VL_OK;
}

void vl_free_liveness(vl_program *p)
{
    // everything below lives in the handle's pools, which are rewound, not freed
    p->live_arena.reset();
    p->tmp_arena.reset();
    p->d_blk_in = p->d_blk_out = p->d_lo_off = p->d_lo = nullptr;
    p->d_opflags = nullptr; p->d_iflags = nullptr;  // (the operand tables live in the layout arena)
    p->d_th_off = p->d_th = p->d_cev_off = nullptr;
    p->d_ev = nullptr;
    p->d_el = nullptr; p->d_el_count = nullptr;
    p->d_ls = p->d_ls_adj = p->d_th_cnt = p->d_blk_th = nullptr;
    p->live_ok = false;
    p->lo_len = 0;
}

extern "C" void vl_program_destroy(vl_program *p)
{
    if (!p) return;
    cudaSetDevice(p->device);
    vl_live_settle(p);
    vl_drop_live_graph(p);
    vl_free_liveness(p);
    if (p->h_live) cudaFreeHost(p->h_live);
    if (p->h_out_pinned) cudaFreeHost(p->h_out_pinned);
    if (p->h_rs) cudaFreeHost(p->h_rs);
    cudaFree(p->d_rs);
    cudaFree(p->d_diag_T);
    cudaFree(p->d_diag_n);
    if (p->ev_live) cudaEventDestroy(p->ev_live);
    p->live_arena.release();
    p->tmp_arena.release();
    p->layout_arena.release();
    cudaFree(p->d_blk_off); cudaFree(p->d_succ_off); cudaFree(p->d_succ); cudaFree(p->d_op_off);
    cudaFree(p->d_ndefs); cudaFree(p->d_op_vreg); cudaFree(p->d_width); cudaFree(p->d_status);
    cudaFree(p->d_bank_list);
    cudaFree(p->d_dict_vreg16); cudaFree(p->d_dict_slotmeta); cudaFree(p->d_dict_opoff); cudaFree(p->d_dict_first4);
    cudaFree(p->d_dict_instr);
    cudaFree(p->d_vcons); cudaFree(p->d_rs_prefix);
    for (auto &v : p->vs) { cudaFree(v.tg); cudaFree(v.cstate); cudaFree(v.anom); cudaFree(v.work); cudaFree(v.racc); cudaFree(v.grp_done); cudaFree(v.thm); }
    for (int j = 0; j < 2; ++j) {
        cudaFree(p->d_stage[j]);
        cudaFree(p->d_stage_out[j]);
        if (p->h_streams[j]) cudaStreamDestroy(p->h_streams[j]);
        if (p->h_events[j]) cudaEventDestroy(p->h_events[j]);
    }
    for (cudaEvent_t ev : p->kt_ev) cudaEventDestroy(ev);
    if (p->ev_fork) cudaEventDestroy(p->ev_fork);
    if (p->ev_pre) cudaEventDestroy(p->ev_pre);
    for (cudaEvent_t ev : p->ev_side)
        if (ev) cudaEventDestroy(ev);
    for (cudaEvent_t ev : p->ev_join)
        if (ev) cudaEventDestroy(ev);
    delete p;
}

// Multiprocessors of a device, asked once per device and process.
int vl_device_sm_count(int device)
{
    static std::atomic<int> cached[64];
    if (device >= 0 && device < 64 && cached[device].load() > 0) return cached[device].load();
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || n <= 0) n = 1;
    if (device >= 0 && device < 64) cached[device].store(n);
    return n;
}

int vl_sm_count(vl_program *p)
{
    if (p->sm_count <= 0) p->sm_count = vl_device_sm_count(p->device);
    return p->sm_count;
}

extern "C" int vl_program_set_option(vl_program *p, int option, uint32_t value)
{
    if (!p) return VL_ERR_INVALID_ARG;
    switch (option) {
    case VL_OPT_CHUNK_INSTRS:
        if (value < 8 || value > 65536) return VL_ERR_INVALID_ARG;
        vl_live_settle(p);
        p->chunk_instrs = value;
        p->live_ok = false;
        return VL_OK;
    case VL_OPT_GROUP:
        if (value != 0 && value != 1 && value != 2 && value != 4 && value != 8) return VL_ERR_INVALID_ARG;
        p->group_opt = value;
        return VL_OK;
    case VL_OPT_SUB_BATCH:
        if (value < 32 || value % 32) return VL_ERR_INVALID_ARG;
        p->sub_batch = value;
        return VL_OK;
    case VL_OPT_KERNEL_TIMING:
        if (value > 1) return VL_ERR_INVALID_ARG;
        p->ktime = (int)value;
        p->kt_used = 0;
        return VL_OK;
    case VL_OPT_LANES:
        if (value < 1 || value > VL_LANES) return VL_ERR_INVALID_ARG;
        p->lanes_opt = value;
        return VL_OK;
    case VL_OPT_PREFETCH_TILES:
        if (value > 64) return VL_ERR_INVALID_ARG;
        p->prefetch_tiles = value;
        return VL_OK;
    case VL_OPT_STAGGER_US:
        if (value > 200) return VL_ERR_INVALID_ARG;
        p->stagger_us = value;
        return VL_OK;
    case VL_OPT_TEST_WAIT:
        if (value > 1) return VL_ERR_INVALID_ARG;
        p->test_wait = value;
        return VL_OK;
    case VL_OPT_THREADS:
        if (value != 0 && value != 256 && value != 512) return VL_ERR_INVALID_ARG;
        p->threads_opt = value;
        return VL_OK;
    default:
        return VL_ERR_INVALID_ARG;
    }
}

extern "C" int vl_program_set_constraints(vl_program *p, const vl_constraints *c)
{
    if (!p) return VL_ERR_INVALID_ARG;
    const uint32_t V = p->V, P = p->P;
    std::vector<uint4> vcons;
    std::vector<uint16_t> prefix;
    uint32_t lo[VL_MAX_CLASSES] = {0}, hi[VL_MAX_CLASSES] = {0};
    hi[0] = P;
    const bool any = c && (c->vreg_align || c->vreg_class || c->reserved_mask);
    if (any) {
        if (c->vreg_class) {
            if (c->n_classes == 0 || c->n_classes > VL_MAX_CLASSES || !c->class_lo || !c->class_hi) return VL_ERR_INVALID_ARG;
            for (uint32_t j = 0; j < c->n_classes; ++j) {
                if (c->class_lo[j] > c->class_hi[j] || c->class_hi[j] > P) return VL_ERR_INVALID_ARG;
                lo[j] = c->class_lo[j];
                hi[j] = c->class_hi[j];
            }
        }
        vcons.resize(V ? V : 1);
        for (uint32_t v = 0; v < V; ++v) {
            const uint32_t al = c->vreg_align ? c->vreg_align[v] : 1u;
            const uint32_t cl = c->vreg_class ? c->vreg_class[v] : 0u;
            if (al == 0 || (c->vreg_class && cl >= c->n_classes)) return VL_ERR_INVALID_ARG;
            vcons[v] = make_uint4(lo[cl] | (hi[cl] << 16), al, al > 1 ? (uint32_t)((0x100000000ull + al - 1) / al) : 0u, 0u);
        }
        if (c->reserved_mask) {
            prefix.resize((size_t)P + 1);
            uint32_t n = 0;
            for (uint32_t r = 0; r < P; ++r) {
                prefix[r] = (uint16_t)n;
                n += (c->reserved_mask[r >> 5] >> (r & 31)) & 1u;
            }
            prefix[P] = (uint16_t)n;  // P <= 65535, so the count fits
        }
    }
    VL_CUDA(p, cudaSetDevice(p->device));
    VL_CUDA(p, cudaDeviceSynchronize());  // verify kernels in flight still read the old rules
    cudaFree(p->d_vcons); p->d_vcons = nullptr;
    cudaFree(p->d_rs_prefix); p->d_rs_prefix = nullptr;
    if (!any) return VL_OK;
    VL_CUDA(p, cudaMalloc(&p->d_vcons, vcons.size() * sizeof(uint4)));
    VL_CUDA(p, cudaMemcpy(p->d_vcons, vcons.data(), vcons.size() * sizeof(uint4), cudaMemcpyHostToDevice));
    if (!prefix.empty()) {
        VL_CUDA(p, cudaMalloc(&p->d_rs_prefix, prefix.size() * sizeof(uint16_t)));
        VL_CUDA(p, cudaMemcpy(p->d_rs_prefix, prefix.data(), prefix.size() * sizeof(uint16_t), cudaMemcpyHostToDevice));
    }
    return VL_OK;
}

extern "C" int vl_liveness(vl_program *p, void *stream)
{
    if (!p) return VL_ERR_INVALID_ARG;
    VL_CUDA(p, cudaSetDevice(p->device));
    // The run goes to an internal stream, behind everything the caller's stream holds now.  The
    // caller's stream does not wait for it: the calls that read the results do (vl_live_join), and
    // the table kernel of a following vl_verify, which needs none of them, runs beside it.
    cudaStream_t *lanes = nullptr;
    int rc = vl_lane_streams(p, &lanes);
    if (rc != VL_OK) return rc;
    cudaStream_t ls = lanes[VL_LIVE_STREAM];
    VL_CUDA(p, cudaEventRecord(p->ev_pre, (cudaStream_t)stream));
    VL_CUDA(p, cudaStreamWaitEvent(ls, p->ev_pre, 0));
    rc = vl_liveness_impl(p, ls);
    p->live_deferred = true;
    return rc;
}

int vl_live_join(vl_program *p, cudaStream_t st)
{
    if (p->live_deferred && p->ev_live) VL_CUDA(p, cudaStreamWaitEvent(st, p->ev_live, 0));
    return VL_OK;
}

extern "C" int vl_liveness_batch(uint32_t n, vl_program *const *progs, void *stream)
{
    if (n == 0) return VL_OK;
    if (!progs) return VL_ERR_INVALID_ARG;
    for (uint32_t j = 0; j < n; ++j)
        if (!progs[j] || progs[j]->device != progs[0]->device) return VL_ERR_INVALID_ARG;
    vl_program *p0 = progs[0];
    VL_CUDA(p0, cudaSetDevice(p0->device));
    cudaStream_t st = (cudaStream_t)stream;
    cudaStream_t *lane = nullptr;
    int rc = vl_lane_streams(p0, &lane);
    if (rc != VL_OK) return rc;
    for (uint32_t j = 0; j < n; ++j) {
        // an earlier single run of one of these programs may still sit on the liveness stream
        if ((rc = vl_live_join(progs[j], st)) != VL_OK) return rc;
        progs[j]->live_deferred = false;
    }
    if (n == 1) return vl_liveness_impl(p0, st);
    VL_CUDA(p0, cudaEventRecord(p0->ev_fork, st));
    for (uint32_t l = 0; l < VL_LANES; ++l) VL_CUDA(p0, cudaStreamWaitEvent(lane[l], p0->ev_fork, 0));
    for (uint32_t j = 0; j < n && rc == VL_OK; ++j) rc = vl_liveness_impl(progs[j], lane[j % VL_LANES]);
    // join even after an error, so that the caller's stream stays ordered after what was launched
    for (uint32_t l = 0; l < VL_LANES; ++l) {
        cudaError_t e = cudaEventRecord(p0->ev_join[l], lane[l]);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, p0->ev_join[l], 0);
        if (e != cudaSuccess && rc == VL_OK) { p0->last_cuda_error = (int)e; rc = VL_ERR_CUDA; }
    }
    return rc;
}

extern "C" int vl_liveness_result(const vl_program *p, const uint32_t **blk_live_in, const uint32_t **blk_live_out,
                                  const uint32_t **lo_off, const uint32_t **lo, uint64_t *lo_len)
{
    if (!p) return VL_ERR_INVALID_ARG;
    if (p->live_pending) {
        const int rc = vl_live_settle(const_cast<vl_program *>(p));
        if (rc != VL_OK) return rc;
    }
    if (!p->live_ok) return VL_ERR_LIVENESS_NOT_RUN;
    if (blk_live_in) *blk_live_in = p->d_blk_in;
    if (blk_live_out) *blk_live_out = p->d_blk_out;
    if (lo_off) *lo_off = p->d_lo_off;
    if (lo) *lo = p->d_lo;
    if (lo_len) *lo_len = p->lo_len;
    return VL_OK;
}

static int check_verify_args(const vl_program *p, const void *cand, uint64_t K, uint64_t pitch, const void *out)
{
    if (!p) return VL_ERR_INVALID_ARG;
    if (!p->live_ok) return VL_ERR_LIVENESS_NOT_RUN;
    if (K == 0) return VL_OK;
    if (!cand || !out) return VL_ERR_INVALID_ARG;
    if (((uintptr_t)cand & 15) || ((uintptr_t)out & 3)) return VL_ERR_INVALID_ARG;
    if (pitch % 8 != 0 || pitch < p->nOp8) return VL_ERR_INVALID_ARG;
    if (K > 0x7FFFFFFFull) return VL_ERR_INVALID_ARG;
    return VL_OK;
}

extern "C" int vl_verify(vl_program *p, const uint16_t *d_cand, uint64_t K, uint64_t pitch, vl_verdict *d_out,
                         void *stream)
{
    int rc = check_verify_args(p, d_cand, K, pitch, d_out);
    if (rc != VL_OK || K == 0) return rc;
    cudaError_t e = cudaSetDevice(p->device);
    if (e != cudaSuccess) return VL_ERR_CUDA;
    rc = vl_verify_lanes(1, &p, &d_cand, &K, &pitch, &d_out, (cudaStream_t)stream);
    // a repeated liveness run may still be in flight: the kernels above are ordered behind it on the
    // stream; its outcome is checked here, after they have been enqueued
    const int rl = vl_live_settle(p);
    return rc != VL_OK ? rc : rl;
}

extern "C" int vl_dict_layout(const vl_program *p, uint32_t *n_entries, const uint32_t **dict_off, const uint32_t **dict_vreg)
{
    if (!p) return VL_ERR_INVALID_ARG;
    if (n_entries) *n_entries = p->nD;
    if (dict_off) *dict_off = p->h_dict_off.data();
    if (dict_vreg) *dict_vreg = p->h_dict_vreg.data();
    return VL_OK;
}

extern "C" int vl_verify_dict(vl_program *p, const uint16_t *d_dict, uint64_t K, uint64_t pitch, vl_verdict *d_out,
                              void *stream)
{
    if (!p) return VL_ERR_INVALID_ARG;
    if (!p->live_ok) return VL_ERR_LIVENESS_NOT_RUN;
    if (K == 0) return VL_OK;
    if (!d_dict || !d_out || ((uintptr_t)d_dict & 15) || ((uintptr_t)d_out & 3)) return VL_ERR_INVALID_ARG;
    if (pitch % 8 != 0 || pitch < p->nD8 || K > 0x7FFFFFFFull) return VL_ERR_INVALID_ARG;
    if (cudaSetDevice(p->device) != cudaSuccess) return VL_ERR_CUDA;
    int rc = vl_verify_lanes(1, &p, &d_dict, &K, &pitch, &d_out, (cudaStream_t)stream, true);
    const int rl = vl_live_settle(p);
    return rc != VL_OK ? rc : rl;
}

extern "C" int vl_verify_batch(uint32_t n, vl_program *const *progs, const uint16_t *const *d_cand,
                               const uint64_t *K, const uint64_t *pitch, vl_verdict *const *d_out, void *stream)
{
    if (n == 0) return VL_OK;
    if (!progs || !d_cand || !K || !pitch || !d_out) return VL_ERR_INVALID_ARG;
    for (uint32_t j = 0; j < n; ++j) {
        int rc = check_verify_args(progs[j], d_cand[j], K[j], pitch[j], d_out[j]);
        if (rc != VL_OK) return rc;
        if (progs[j]->device != progs[0]->device) return VL_ERR_INVALID_ARG;
    }
    if (cudaSetDevice(progs[0]->device) != cudaSuccess) return VL_ERR_CUDA;
    uint32_t first = 0;  // the first program with rows lends its fork / join events
    while (first < n && K[first] == 0) ++first;
    if (first == n) return VL_OK;
    int rc = vl_verify_lanes(n - first, progs + first, d_cand + first, K + first, pitch + first, d_out + first,
                             (cudaStream_t)stream);
    for (uint32_t j = 0; j < n; ++j) {
        const int rl = vl_live_settle(progs[j]);
        if (rc == VL_OK) rc = rl;
    }
    return rc;
}

extern "C" int vl_verify_host(vl_program *p, const uint16_t *h_cand, uint64_t K, uint64_t pitch, vl_verdict *h_out,
                              void *stream)
{
    int rc = check_verify_args(p, h_cand, K, pitch, h_out);
    if (rc != VL_OK || K == 0) return rc;
    VL_CUDA(p, cudaSetDevice(p->device));
    if ((rc = vl_live_settle(p)) != VL_OK) return rc;
    // slabs of about 64 MiB, a multiple of 4 rows
    uint64_t rows = std::max<uint64_t>(4, ((64ull << 20) / (pitch * 2)) / 4 * 4);
    rows = std::min<uint64_t>(rows, (K + 3) / 4 * 4);
    if (p->stage_rows < rows || p->stage_pitch != pitch) {
        for (int j = 0; j < 2; ++j) {
            cudaFree(p->d_stage[j]); cudaFree(p->d_stage_out[j]);
            p->d_stage[j] = nullptr; p->d_stage_out[j] = nullptr;
        }
        p->stage_rows = 0;
        for (int j = 0; j < 2; ++j) {
            VL_CUDA(p, cudaMalloc((void **)&p->d_stage[j], rows * pitch * 2));
            VL_CUDA(p, cudaMalloc((void **)&p->d_stage_out[j], rows * sizeof(vl_verdict)));
        }
        p->stage_rows = rows;
        p->stage_pitch = pitch;
    }
    rows = p->stage_rows;
    for (int j = 0; j < 2; ++j) {
        if (!p->h_streams[j]) VL_CUDA(p, cudaStreamCreateWithFlags(&p->h_streams[j], cudaStreamNonBlocking));
        if (!p->h_events[j]) VL_CUDA(p, cudaEventCreateWithFlags(&p->h_events[j], cudaEventDisableTiming));
    }
    // The verdicts come back through pinned memory of the handle: a copy straight into pageable
    // caller memory would make every slab wait for its kernels before the next slab's rows are sent.
    if (p->h_out_cap < K) {
        if (p->h_out_pinned) cudaFreeHost(p->h_out_pinned);
        p->h_out_pinned = nullptr;
        p->h_out_cap = 0;
        VL_CUDA(p, cudaHostAlloc((void **)&p->h_out_pinned, K * sizeof(vl_verdict), cudaHostAllocDefault));
        p->h_out_cap = K;
    }
    VL_CUDA(p, cudaEventRecord(p->h_events[0], (cudaStream_t)stream));
    for (int j = 0; j < 2; ++j) VL_CUDA(p, cudaStreamWaitEvent(p->h_streams[j], p->h_events[0], 0));
    uint64_t slab = 0;
    for (uint64_t k0 = 0; k0 < K; k0 += rows, ++slab) {
        int j = (int)(slab & 1);
        uint64_t n = std::min(rows, K - k0);
        VL_CUDA(p, cudaMemcpyAsync(p->d_stage[j], h_cand + k0 * pitch, n * pitch * 2, cudaMemcpyHostToDevice,
                                   p->h_streams[j]));
        rc = vl_verify_impl(p, p->d_stage[j], n, pitch, p->d_stage_out[j], p->h_streams[j], VL_LANES + j);
        if (rc != VL_OK) return rc;
        VL_CUDA(p, cudaMemcpyAsync(p->h_out_pinned + k0, p->d_stage_out[j], n * sizeof(vl_verdict),
                                   cudaMemcpyDeviceToHost, p->h_streams[j]));
    }
    for (int j = 0; j < 2; ++j) VL_CUDA(p, cudaStreamSynchronize(p->h_streams[j]));
    memcpy(h_out, p->h_out_pinned, K * sizeof(vl_verdict));
    return VL_OK;
}

extern "C" int vl_verify_status(vl_program *p, void *stream)
{
    if (!p) return VL_ERR_INVALID_ARG;
    VL_CUDA(p, cudaSetDevice(p->device));
    uint32_t st = 0;
    VL_CUDA(p, cudaMemcpyAsync(&st, p->d_status + 1, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    VL_CUDA(p, cudaMemsetAsync(p->d_status + 1, 0, 4, (cudaStream_t)stream));
    VL_CUDA(p, cudaStreamSynchronize((cudaStream_t)stream));
    return (st & ST_DEVICE_WAIT) ? VL_ERR_DEVICE_WAIT : VL_OK;
}

extern "C" uint64_t vl_kernel_launches(void) { return g_vl_launches.load(); }

extern "C" int vl_kernel_times(vl_program *p, float ms[4], uint32_t *passes)
{
    if (!p || !ms) return VL_ERR_INVALID_ARG;
    for (int j = 0; j < 4; ++j) ms[j] = 0.f;
    const size_t n = p->kt_used / 5;
    if (passes) *passes = (uint32_t)n;
    if (n) {
        cudaSetDevice(p->device);
        VL_CUDA(p, cudaEventSynchronize(p->kt_ev[n * 5 - 1]));
        for (size_t i = 0; i < n; ++i)
            for (int j = 0; j < 4; ++j) {
                float t = 0.f;
                VL_CUDA(p, cudaEventElapsedTime(&t, p->kt_ev[i * 5 + j], p->kt_ev[i * 5 + j + 1]));
                ms[j] += t;
            }
    }
    p->kt_used = 0;
    return VL_OK;
}

extern "C" int vl_last_cuda_error(const vl_program *p) { return p ? p->last_cuda_error : 0; }

extern "C" const char *vl_strerror(int code)
{
    switch (code) {
    case VL_OK: return "ok";
    case VL_ERR_INVALID_ARG: return "invalid argument";
    case VL_ERR_MALFORMED_PROGRAM: return "malformed program";
    case VL_ERR_NOT_STRICT: return "program is not strict: a virtual register is live into the entry block";
    case VL_ERR_LIVENESS_NOT_RUN: return "vl_liveness has not been run on this program";
    case VL_ERR_UNSUPPORTED: return "program exceeds what the kernels support";
    case VL_ERR_NO_CONVERGE: return "liveness did not converge";
    case VL_ERR_CUDA: return "CUDA call failed";
    case VL_ERR_DEVICE_WAIT: return "a bounded wait inside a kernel ran out";
    default: return "unknown error";
    }
}
