// C-ABI of the isomorphic neighbourhood collectives (declared in include/iso.h):
// argument checking, object lifetime, device tables and kernel launches.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <mutex>
#include <vector>

#include "iso.h"
#include "iso_internal.h"
#include "iso_kernels.cuh"

using namespace iso;

struct Iso_comm_s : public Comm {};
struct Iso_request_s : public Request {};

namespace {

thread_local int g_last_cuda_error = 0;

int cuda_fail(cudaError_t e)
{
    g_last_cuda_error = (int)e;
    (void)cudaGetLastError();  // clear the sticky flag of non-fatal errors
    return e == cudaErrorMemoryAllocation ? ISO_ERR_NOMEM : ISO_ERR_CUDA;
}

#define ISO_CUDA(call)                               \
    do {                                             \
        cudaError_t e_ = (call);                     \
        if (e_ != cudaSuccess) return cuda_fail(e_); \
    } while (0)

void release_device(Request &r)
{
    if (r.graph_exec) cudaGraphExecDestroy(static_cast<cudaGraphExec_t>(r.graph_exec));
    r.graph_exec = nullptr;
    if (r.host_graph_exec) cudaGraphExecDestroy(static_cast<cudaGraphExec_t>(r.host_graph_exec));
    r.host_graph_exec = nullptr;
    r.host_last_hs = r.host_last_hr = nullptr;
    if (r.host_main_stream) cudaStreamDestroy(static_cast<cudaStream_t>(r.host_main_stream));
    r.host_main_stream = nullptr;
    if (r.d_blob) cudaFree(r.d_blob);
    if (r.d_inter_alloc) cudaFree(r.d_inter_alloc);
    r.d_inter_alloc = nullptr;
    if (r.d_err) cudaFree(r.d_err);
    for (void *st : r.host_streams) cudaStreamDestroy(static_cast<cudaStream_t>(st));
    r.host_streams.clear();
    for (void *e : r.slab_events) cudaEventDestroy(static_cast<cudaEvent_t>(e));
    for (void *e : r.host_timing) cudaEventDestroy(static_cast<cudaEvent_t>(e));
    r.host_timing.clear();
    r.host_timed = false;
    r.slab_events.clear();
    if (r.d_counter) cudaFree(r.d_counter);
    r.d_counter = nullptr;
    r.wave_counters = 0;
    r.multi_grid = 0;
    r.wave_grid = 0;
    if (r.h_err) cudaFreeHost(r.h_err);
    r.d_blob = nullptr;
    r.d_inter = nullptr;
    r.d_err = nullptr;
    r.h_err = nullptr;
    r.d_inter_bytes = 0;
    r.dirty = true;
}

void comm_unref(Comm *c)
{
    if (c && --c->refcount == 0) delete static_cast<Iso_comm_s *>(c);
}

bool mul_overflows(int64_t a, int64_t b)
{
    if (a == 0 || b == 0) return false;
    return a > INT64_MAX / b;
}

// Common tail of the init calls: strides are set, block layout is in r.
int finish_init(Iso_request_s *r, Iso_request *out)
{
    const Comm &c = *r->comm;
    if (mul_overflows(c.P, r->send_stride) || mul_overflows(c.P, r->recv_stride)) {
        comm_unref(r->comm);
        delete r;
        return ISO_ERR_COUNT;
    }
    // receive blocks must not overlap each other
    {
        std::vector<std::pair<int64_t, int64_t>> iv;
        for (int i = 0; i < r->s; ++i)
            if (r->len[i] > 0) iv.push_back({r->rdispl[i], r->rdispl[i] + r->len[i]});
        std::sort(iv.begin(), iv.end());
        for (size_t k = 1; k < iv.size(); ++k)
            if (iv[k].first < iv[k - 1].second) {
                comm_unref(r->comm);
                delete r;
                return ISO_ERR_OVERLAP;
            }
    }
    // the two user buffers must not overlap
    if (r->send && r->recv) {
        const unsigned char *s0 = r->send, *s1 = r->send + c.P * r->send_stride;
        const unsigned char *d0 = r->recv, *d1 = r->recv + c.P * r->recv_stride;
        if (s0 < d1 && d0 < s1 && s0 != s1 && d0 != d1) {
            comm_unref(r->comm);
            delete r;
            return ISO_ERR_OVERLAP;
        }
    }
    int rc = build_schedule(*r);
    if (rc == ISO_SUCCESS) rc = lower_schedule(*r, (uintptr_t)r->send, (uintptr_t)r->recv, 0);
    if (rc != ISO_SUCCESS) {
        comm_unref(r->comm);
        delete r;
        return rc;
    }
    *out = r;
    return ISO_SUCCESS;
}

Iso_request_s *new_request(Iso_comm comm, int kind, const void *sendbuf, void *recvbuf)
{
    Iso_request_s *r = new (std::nothrow) Iso_request_s();
    if (!r) return nullptr;
    r->comm = comm;
    comm->refcount++;
    r->kind = kind;
    r->knobs = read_knobs();
    if (r->knobs.sender_side >= 0 && r->knobs.sender_side <= 2) r->sender_side = r->knobs.sender_side;
    if (r->knobs.hybrid >= 0) r->hybrid = r->knobs.hybrid != 0;
    default_dimension_order(*r);
    r->send = static_cast<const unsigned char *>(sendbuf);
    r->recv = static_cast<unsigned char *>(recvbuf);
    r->s = comm->s;
    r->len.assign(comm->s, 0);
    r->sdispl.assign(comm->s, 0);
    r->rdispl.assign(comm->s, 0);
    return r;
}

int64_t round_up16(int64_t x) { return (x + 15) / 16 * 16; }

// Guard bands around the library's intermediate buffer (a multiple of 256 bytes, so that the
// buffer keeps the allocation's alignment).
constexpr size_t kGuardBytes = 4096;
constexpr int kGuardPattern = 0xC3;

LaunchDev make_launch_args(const Request &r, const LaunchPlan &L);
void choose_slab_plan(Request &r);
int build_wave(Request &r, unsigned char *blob, size_t launches_off, size_t items_off, size_t slabs);

// One descriptor per unit position of a vector launch: parts in their order, the units of
// a part in address order.
void fill_units(const Request &r, const LaunchPlan &L, UnitDev *ud)
{
    const Comm &c = *r.comm;
    const int64_t stride[3] = {r.send_stride, r.recv_stride, r.inter_stride};
    int used_index[ISO_MAX_DIMS];
    for (int j = 0; j < ISO_MAX_DIMS; ++j) used_index[j] = -1;
    for (int k = 0; k < L.n_used; ++k) used_index[L.used_dim[k]] = k;
    std::vector<UnitDev> units(L.units_per_proc);
    for (const LoweredPart &lp : L.parts) {
        UnitDev u{};
        long long delta = 0;
        if (!L.compact) {
            u.nnz = (uint8_t)L.n_used;
            for (int z = 0; z < L.n_used; ++z) u.dim[z] = (uint8_t)z;
        }
        for (int j = 0; j < c.d; ++j) {
            // periodic dimension: the shift (wrap test); mesh dimension: the check value
            const int value = c.periodic[j] ? lp.p.shift[j] : lp.p.check[j];
            delta -= (long long)lp.p.shift[j] * c.rank_stride[j];
            if (!value) continue;
            if (L.compact) {
                u.dim[u.nnz] = (uint8_t)used_index[j];
                u.c[u.nnz++] = value;
            } else {
                u.c[used_index[j]] = value;
            }
        }
        u.src_buf = (uint8_t)lp.p.src_buf;
        u.dst_buf = (uint8_t)lp.p.dst_buf;
        u.width = (uint8_t)lp.width;
        for (uint32_t k = 0; k < lp.units; ++k) {
            u.src_term = delta * stride[lp.p.src_buf] + lp.p.src_off + (int64_t)k * lp.width;
            u.dst_term = lp.p.dst_off + (int64_t)k * lp.width;
            units[lp.first_unit + k] = u;
        }
    }
    std::copy(units.begin(), units.end(), ud);
}

// Descriptors of a sender-side launch: one per 16-byte unit of every parent block.
void fill_fans(const Request &r, const LaunchPlan &L, FanDev *fd)
{
    const Comm &c = *r.comm;
    const int64_t stride[3] = {r.send_stride, r.recv_stride, r.inter_stride};
    const int64_t rank_stride = L.n_used ? c.rank_stride[L.used_dim[0]] : 0;
    size_t at = 0;
    for (const FanParent &f : L.fans) {
        FanDev d{};
        d.src_buf = (uint8_t)f.src_buf;
        d.n_dst = (uint8_t)f.dsts.size();
        for (int64_t k = 0; k < f.len / 16; ++k) {
            d.src_term = f.src_off + 16 * k;
            for (size_t e = 0; e < f.dsts.size(); ++e) {
                d.dst_buf[e] = (uint8_t)f.dsts[e].buf;
                d.c[e] = f.dsts[e].c;
                d.dst_term[e] = f.dsts[e].off + 16 * k + (int64_t)f.dsts[e].c * rank_stride * stride[f.dsts[e].buf];
            }
            fd[at++] = d;
        }
    }
}

// Uploads the lowered schedule and allocates the intermediate buffer.
int materialise(Request &r)
{
    const Comm &c = *r.comm;
    // a captured graph holds the addresses of the tables and buffers that are replaced below
    if (r.graph_exec) cudaGraphExecDestroy(static_cast<cudaGraphExec_t>(r.graph_exec));
    r.graph_exec = nullptr;
    if (r.host_graph_exec) cudaGraphExecDestroy(static_cast<cudaGraphExec_t>(r.host_graph_exec));
    r.host_graph_exec = nullptr;
    r.host_last_hs = r.host_last_hr = nullptr;
    // grids are sized for the device that runs them (the host-only lowering at init assumed a B200)
    int device = 0, sms = 0;
    ISO_CUDA(cudaGetDevice(&device));
    ISO_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    if (sms > 0) r.sm_count = sms;
    {
        // lowered afresh with the request's present settings: the slab plan below reads it
        int rc0 = lower_schedule(r, (uintptr_t)r.send, (uintptr_t)r.recv, (uintptr_t)r.d_inter);
        if (rc0 != ISO_SUCCESS) return rc0;
    }
    // pipelined one-launch execution: every launch must be a 16-byte vector launch of at most
    // 256 threads on periodic dimensions.  Decided on a trial lowering (device allocations
    // are 256-byte aligned) because the size of the intermediate buffer depends on it.
    r.wave_ok = false;
    r.wave_grid = 0;
    r.wave_slabs = 0;
    if (r.wave_request > 0) {
        int rc0 = lower_schedule(r, (uintptr_t)r.send, (uintptr_t)r.recv, 0);
        if (rc0 != ISO_SUCCESS) return rc0;
        bool ok = !r.launches.empty();
        for (const LaunchPlan &L : r.launches) {
            if (L.kernel != KERNEL_VEC || L.width != 16 || L.threads > 1024) ok = false;
            for (int k = 0; k < L.n_used; ++k)
                if (!c.periodic[L.used_dim[k]]) ok = false;
        }
        r.wave_ok = ok;
    }
    choose_slab_plan(r);
    // device tables depend on the alignment of the intermediate buffer: allocate it first
    const int64_t inter_bytes = r.inter_rows * r.inter_stride;
    if (inter_bytes != r.d_inter_bytes) {  // exactly sized, so that the trailing band sits right behind it
        if (r.d_inter_alloc) cudaFree(r.d_inter_alloc);
        r.d_inter = r.d_inter_alloc = nullptr;
        r.d_inter_bytes = 0;
        // a guard band of a fixed pattern on either side: no schedule may ever write there
        // (Iso_request_check_guards)
        if (inter_bytes > 0) {
        ISO_CUDA(cudaMalloc((void **)&r.d_inter_alloc, (size_t)inter_bytes + 2 * kGuardBytes));
        r.d_inter = r.d_inter_alloc + kGuardBytes;
        r.d_inter_bytes = inter_bytes;
        ISO_CUDA(cudaMemset(r.d_inter_alloc, kGuardPattern, kGuardBytes));
        ISO_CUDA(cudaMemset(r.d_inter + inter_bytes, kGuardPattern, kGuardBytes));
        }
    }
    int rc = lower_schedule(r, (uintptr_t)r.send, (uintptr_t)r.recv, (uintptr_t)r.d_inter);
    if (rc != ISO_SUCCESS) return rc;

    // every plan that needs tables: the launches and the bulk sides of hybrid launches
    std::vector<LaunchPlan *> plans;
    for (LaunchPlan &L : r.launches) {
        plans.push_back(&L);
        for (LaunchPlan &S : L.side) plans.push_back(&S);
    }
    size_t bytes = 0;
    for (LaunchPlan *plan : plans) {
        LaunchPlan &L = *plan;
        L.parts_off = bytes;
        bytes += L.parts.size() * sizeof(PartDev);
        L.lookup_off = bytes;
        bytes += (L.lookup.size() * sizeof(uint16_t) + 15) / 16 * 16;
        L.units_off = bytes;
        if (L.kernel == KERNEL_VEC) bytes += (size_t)L.units_per_proc * sizeof(UnitDev);
        if (L.kernel == KERNEL_FAN) bytes += (size_t)L.units_per_proc * sizeof(FanDev);
    }
    // one-launch execution: every launch is a 16-byte vector launch on periodic dimensions
    bool single = r.persistent && !r.wave_ok && r.launches.size() >= 2;
    for (const LaunchPlan &L : r.launches) {
        if (L.kernel != KERNEL_VEC || L.width != 16 || L.threads > 1024) single = false;
        for (int k = 0; k < L.n_used; ++k)
            if (!c.periodic[L.used_dim[k]]) single = false;
    }
    bytes = (bytes + 127) / 128 * 128;
    const size_t launches_off = bytes;
    if (single) bytes += r.launches.size() * sizeof(LaunchDev);
    // pipelined one-launch execution: one descriptor and one item record per (slab, launch)
    const size_t wave_slabs = r.wave_ok ? std::max<size_t>(1, r.slab_plan.size()) : 0;
    const size_t wave_n = wave_slabs * r.launches.size();
    bytes = (bytes + 127) / 128 * 128;
    const size_t wave_launches_off = bytes;
    bytes += wave_n * sizeof(LaunchDev);
    bytes = (bytes + 127) / 128 * 128;
    const size_t wave_items_off = bytes;
    bytes += wave_n * sizeof(WaveItem);
    std::vector<unsigned char> blob(bytes ? bytes : 16, 0);
    for (const LaunchPlan *plan : plans) {
        const LaunchPlan &L = *plan;
        int used_index[ISO_MAX_DIMS];
        for (int j = 0; j < ISO_MAX_DIMS; ++j) used_index[j] = -1;
        for (int k = 0; k < L.n_used; ++k) used_index[L.used_dim[k]] = k;
        PartDev *pd = reinterpret_cast<PartDev *>(blob.data() + L.parts_off);
        for (size_t t = 0; t < L.parts.size(); ++t) {
            const LoweredPart &lp = L.parts[t];
            PartDev d{};
            d.src_off = lp.p.src_off;
            d.dst_off = lp.p.dst_off;
            d.len = lp.p.len;
            d.first_unit = lp.first_unit;
            d.units = lp.units;
            d.src_buf = (uint8_t)lp.p.src_buf;
            d.dst_buf = (uint8_t)lp.p.dst_buf;
            long long delta = 0;
            int nnz = 0;
            for (int j = 0; j < c.d; ++j) {
                // periodic dimension: the shift (wrap test); mesh dimension: the check value
                const int value = c.periodic[j] ? lp.p.shift[j] : lp.p.check[j];
                delta -= (long long)lp.p.shift[j] * c.rank_stride[j];
                if (!value) continue;
                d.dim[nnz] = (uint8_t)used_index[j];
                d.c[nnz] = value;
                ++nnz;
            }
            d.nnz = (uint8_t)nnz;
            d.rank_delta = delta;
            pd[t] = d;
        }
        if (!L.lookup.empty())
            std::memcpy(blob.data() + L.lookup_off, L.lookup.data(), L.lookup.size() * sizeof(uint16_t));
        if (L.kernel == KERNEL_VEC) fill_units(r, L, reinterpret_cast<UnitDev *>(blob.data() + L.units_off));
        if (L.kernel == KERNEL_FAN) fill_fans(r, L, reinterpret_cast<FanDev *>(blob.data() + L.units_off));
    }
    if (r.d_blob) cudaFree(r.d_blob);
    r.d_blob = nullptr;
    ISO_CUDA(cudaMalloc(&r.d_blob, blob.size()));
    r.multi_grid = 0;
    if (single || wave_n > 0) {
        const int need = (int)std::max<size_t>(1, wave_n);
        if (!r.d_counter || r.wave_counters < need) {
            if (r.d_counter) cudaFree(r.d_counter);
            r.d_counter = nullptr;
            ISO_CUDA(cudaMalloc((void **)&r.d_counter, (size_t)need * sizeof(unsigned long long)));
            r.wave_counters = need;
        }
        // a changed plan counts afresh
        ISO_CUDA(cudaMemset(r.d_counter, 0, (size_t)r.wave_counters * sizeof(unsigned long long)));
        r.epoch = 0;
        r.wave_run = 0;
    }
    if (wave_n > 0) {
        int rcw = build_wave(r, blob.data(), wave_launches_off, wave_items_off, wave_slabs);
        if (rcw != ISO_SUCCESS) return rcw;
    }
    if (single) {
        // the grid must be resident as a whole: ask how many CTAs fit
        const size_t smem = (sizeof(LaunchDev) + 127) / 128 * 128 + (size_t)kWideDepth * 1024 * 16;
        ISO_CUDA(cudaFuncSetAttribute(iso_gather_rows_multi<kWideDepth>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        int per_sm = 0;
        ISO_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, iso_gather_rows_multi<kWideDepth>, 1024, smem));
        int want = 4;
        if (r.knobs.vec_ctas_per_sm >= 1 && r.knobs.vec_ctas_per_sm <= 8) want = r.knobs.vec_ctas_per_sm;
        per_sm = std::min(per_sm, want);
        if (per_sm >= 1) {
            r.multi_grid = per_sm * r.sm_count;
            r.multi_smem = smem;
            r.multi_launches_off = launches_off;
            LaunchDev *ld = reinterpret_cast<LaunchDev *>(blob.data() + launches_off);
            for (size_t k = 0; k < r.launches.size(); ++k) ld[k] = make_launch_args(r, r.launches[k]);
        }
    }
    ISO_CUDA(cudaMemcpy(r.d_blob, blob.data(), blob.size(), cudaMemcpyHostToDevice));
    if (!r.d_err) {
        ISO_CUDA(cudaMalloc((void **)&r.d_err, sizeof(int)));
        ISO_CUDA(cudaMemset(r.d_err, 0, sizeof(int)));
    }
    if (!r.h_err) {
        ISO_CUDA(cudaMallocHost((void **)&r.h_err, sizeof(int)));
        *r.h_err = 0;
    }
    // opt in to large dynamic shared memory once per kernel and device
    {
        static std::vector<int> devices_set;
        static std::mutex guard;
        std::lock_guard<std::mutex> lock(guard);
        if (std::find(devices_set.begin(), devices_set.end(), device) == devices_set.end()) {
            ISO_CUDA(cudaFuncSetAttribute(iso_gather_bulk, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            devices_set.push_back(device);
        }
    }
    r.dirty = false;
    return ISO_SUCCESS;
}

LaunchDev make_launch_args(const Request &r, const LaunchPlan &L)
{
    const Comm &c = *r.comm;
    LaunchDev a{};
    a.parts = reinterpret_cast<const PartDev *>(static_cast<unsigned char *>(r.d_blob) + L.parts_off);
    a.lookup = reinterpret_cast<const uint16_t *>(static_cast<unsigned char *>(r.d_blob) + L.lookup_off);
    a.units = reinterpret_cast<const UnitDev *>(static_cast<unsigned char *>(r.d_blob) + L.units_off);
    a.buf[ISO_BUF_SEND] = const_cast<unsigned char *>(r.send);
    a.buf[ISO_BUF_RECV] = r.recv;
    a.buf[ISO_BUF_INTER] = r.d_inter;
    a.buf_stride[ISO_BUF_SEND] = r.send_stride;
    a.buf_stride[ISO_BUF_RECV] = r.recv_stride;
    a.buf_stride[ISO_BUF_INTER] = r.inter_stride;
    a.P = c.P;
    a.row_lo = 0;
    a.row_hi = c.P;
    a.err = r.d_err;
    a.nparts = (uint32_t)L.parts.size();
    a.units_per_proc = L.units_per_proc;
    a.uniform_units = L.uniform_units;
    a.lookup_shift = (uint32_t)L.lookup_shift;
    a.width = (uint32_t)L.width;
    a.chunk_units = L.chunk_units;
    a.rows_per_pass = L.rows_per_pass;
    a.tile_procs = L.tile_procs;
    // Slab execution with many slabs: one slab's intermediate blocks are a small part of the L2
    // and are recycled every few tens of microseconds; kept resident (evict_last) they are no
    // longer written back before the next slab overwrites them.  Measured with the hint against
    // without: 4 KB blocks in 128 slabs 3.00 against 3.15 ms, 512-byte blocks in 16 slabs 362
    // against 393 microseconds, shells in 32 slabs 2.63 against 2.84 ms, Moore r=3 in 16 slabs 540
    // against 547; with few slabs the kept lines crowd out the streamed ones: 8 slabs (16^4 torus)
    // 284 against 281, 2 slabs (8^5 torus) 158 against 155, no slabs (32^3 torus) 38.6 against 37.1.
    a.keep_inter = (r.knobs.l2_keep && r.slab_plan.size() >= 16) ? 1u : 0u;
    a.n_used = L.n_used;
    a.mesh_mask = 0;
    a.grid_share = 1;
    a.col_split = (uint32_t)L.col_split;
    FastDiv f = make_fastdiv(L.units_per_proc);
    a.div_units = FastDivDev{f.m, f.s1, f.s2, f.div};
    f = make_fastdiv(L.uniform_units ? L.uniform_units : 1);
    a.div_uniform = FastDivDev{f.m, f.s1, f.s2, f.div};
    for (int k = 0; k < L.n_used; ++k) {
        const int j = L.used_dim[k];
        a.used_dim[k] = j;
        a.used_size[k] = (uint32_t)c.dims[j];
        a.used_rstride[k] = c.rank_stride[j];
        a.used_wrap[k] = (uint32_t)(c.dims[j] * c.rank_stride[j]);
        f = make_fastdiv((uint32_t)c.rank_stride[j]);
        a.div_rstride[k] = FastDivDev{f.m, f.s1, f.s2, f.div};
        f = make_fastdiv((uint32_t)c.dims[j]);
        a.div_size[k] = FastDivDev{f.m, f.s1, f.s2, f.div};
        if (!c.periodic[j]) a.mesh_mask |= 1 << k;
    }
    return a;
}

// Item list of the pipelined one-launch execution.  Slabs are taken two at a time and
// their launches interleaved: (a, l0), (b, l0), (a, l1), (b, l1), ... so that between an
// item and the one it waits for lies an item of the other slab.  With three or more slabs
// the intermediate buffer holds two slabs (even and odd ones alternate between the halves).
// An item waits for the latest of: the launches of earlier phases on its own slab, and -
// if it writes intermediate places - every launch of the slab that used its half before.
int build_wave(Request &r, unsigned char *blob, size_t launches_off, size_t items_off, size_t n_slabs)
{
    const Comm &c = *r.comm;
    const size_t nl = r.launches.size();
    const size_t n = n_slabs * nl;
    const size_t smem = (sizeof(LaunchDev) + 127) / 128 * 128 + (size_t)kWideDepth * 1024 * 16;
    ISO_CUDA(cudaFuncSetAttribute(iso_gather_rows_wave<kWideDepth>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int per_sm = 0;
    ISO_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, iso_gather_rows_wave<kWideDepth>, 1024, smem));
    int want = 4;
    if (r.knobs.vec_ctas_per_sm >= 1 && r.knobs.vec_ctas_per_sm <= 8) want = r.knobs.vec_ctas_per_sm;
    per_sm = std::min(per_sm, want);
    if (per_sm < 1) return ISO_SUCCESS;  // cannot be resident: Iso_Start falls back to one launch per phase
    const int grid = per_sm * r.sm_count;

    std::vector<std::pair<long long, long long>> slabs = r.slab_plan;
    if (slabs.empty()) slabs.push_back({0, c.P});
    long long slab_rows = 0;
    for (const auto &w : slabs) slab_rows = std::max(slab_rows, w.second - w.first);
    const bool halves = slabs.size() >= 3;

    LaunchDev *ld = reinterpret_cast<LaunchDev *>(blob + launches_off);
    WaveItem *items = reinterpret_cast<WaveItem *>(blob + items_off);
    std::vector<int> index_of(n, -1);        // (slab, launch) -> item
    std::vector<int> last_of_slab(slabs.size(), -1);
    std::vector<char> writes_inter(nl, 0);
    for (size_t l = 0; l < nl; ++l)
        for (const LoweredPart &lp : r.launches[l].parts)
            if (lp.p.dst_buf == ISO_BUF_INTER) writes_inter[l] = 1;
    size_t i = 0;
    unsigned long long groups_so_far = 0;
    for (size_t k0 = 0; k0 < slabs.size(); k0 += 2) {
        const size_t k1 = std::min(slabs.size(), k0 + 2);
        for (size_t l = 0; l < nl; ++l)
            for (size_t k = k0; k < k1; ++k) {
                const LaunchPlan &L = r.launches[l];
                LaunchDev a = make_launch_args(r, L);
                a.row_lo = slabs[k].first;
                a.row_hi = slabs[k].second;
                if (halves && a.buf[ISO_BUF_INTER])
                    a.buf[ISO_BUF_INTER] -= (slabs[k].first - (long long)(k & 1) * slab_rows) * r.inter_stride;
                ld[i] = a;
                WaveItem it{};
                it.wait_item = -1;
                for (size_t l2 = 0; l2 < nl; ++l2)
                    if (r.launches[l2].phase < L.phase && index_of[k * nl + l2] >= 0)
                        it.wait_item = std::max(it.wait_item, index_of[k * nl + l2]);
                if (halves && writes_inter[l] && k >= 2) it.wait_item = std::max(it.wait_item, last_of_slab[k - 2]);
                it.cta_offset = (uint32_t)(groups_so_far % (unsigned long long)grid);
                const int count = L.compact ? L.max_nnz : L.n_used;
                it.variant = L.compact ? (count <= 3 ? 4 + std::max(1, count) : 8) : (count <= 3 ? count : 4);
                items[i] = it;
                index_of[k * nl + l] = (int)i;
                last_of_slab[k] = (int)i;
                groups_so_far += (unsigned long long)((a.row_hi - a.row_lo + L.rows_per_pass - 1) / L.rows_per_pass);
                ++i;
            }
    }
    r.wave_grid = grid;
    r.wave_items = (int)n;
    r.wave_smem = smem;
    r.wave_launches_off = launches_off;
    r.wave_items_off = items_off;
    r.wave_slabs = (int)slabs.size();
    return ISO_SUCCESS;
}

// Grid for the rows [a.row_lo, a.row_hi): the plan's grid scaled to the share of the rows.
unsigned grid_for_rows(const LaunchPlan &L, const LaunchDev &a, int share = 1)
{
    const long long rows = a.row_hi - a.row_lo;
    if (rows >= a.P && share <= 1) return (unsigned)L.grid;
    if (L.kernel == KERNEL_BULK) return (unsigned)((rows + a.tile_procs - 1) / a.tile_procs);
    const long long groups = (rows + L.rows_per_pass - 1) / L.rows_per_pass;
    // `share` launches of this kind run side by side: each takes its part of the CTA slots
    const long long full = std::max<long long>(1, L.grid / std::max(1, share));
    if (L.col_split > 1)  // CTAs per column chunk x chunks
        return (unsigned)(std::max<long long>(1, std::min<long long>(full / L.col_split, groups)) * L.col_split);
    const long long g = std::max<long long>(1, std::min<long long>(full, groups));
    return (unsigned)g;
}

constexpr int kMaxDynamicSmem = 227 * 1024;  // dynamic shared memory a CTA can opt in to on sm_100

// Shared memory of a wide launch that keeps a coordinate table behind the cp.async ring.
size_t table_bytes(const LaunchDev &a) { return (size_t)a.tab_iters * a.rows_per_pass * a.tab_stride * sizeof(uint32_t); }

template <typename Kernel>
cudaError_t launch_kernel(Kernel kernel, const LaunchPlan &L, const LaunchDev &a, cudaStream_t stream, bool dependent)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid_for_rows(L, a, a.grid_share));
    cfg.blockDim = dim3((unsigned)L.threads);
    cfg.dynamicSmemBytes = L.smem + table_bytes(a);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    // programmatic dependent launch: the kernel may start while its predecessor in the stream
    // drains; it orders itself behind it with griddepcontrol.wait before touching data
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, a);
}

// Wide CTAs need more dynamic shared memory than the default limit: opt in once per kernel.
template <typename Kernel>
cudaError_t launch_wide(Kernel kernel, const LaunchPlan &L, const LaunchDev &a, cudaStream_t stream, bool dependent)
{
    // (device, kernel) pairs that already have the larger limit: the attribute is per device
    static std::vector<std::pair<int, const void *>> opted_in;
    static std::mutex guard;
    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return e;
    const std::pair<int, const void *> key(device, reinterpret_cast<const void *>(kernel));
    {
        std::lock_guard<std::mutex> lock(guard);
        if (std::find(opted_in.begin(), opted_in.end(), key) == opted_in.end()) {
            e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem);
            if (e != cudaSuccess) return e;
            opted_in.push_back(key);
        }
    }
    return launch_kernel(kernel, L, a, stream, dependent);
}

// The hybrid kernel: the vector side's threads plus one warp for the bulk side.
template <typename Kernel>
cudaError_t launch_hybrid(Kernel kernel, const LaunchPlan &L, const LaunchDev &a, const LaunchDev &side, size_t smem,
                          cudaStream_t stream, bool dependent)
{
    static std::vector<std::pair<int, const void *>> opted_in;
    static std::mutex guard;
    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return e;
    const std::pair<int, const void *> key(device, reinterpret_cast<const void *>(kernel));
    {
        std::lock_guard<std::mutex> lock(guard);
        if (std::find(opted_in.begin(), opted_in.end(), key) == opted_in.end()) {
            e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem);
            if (e != cudaSuccess) return e;
            opted_in.push_back(key);
        }
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid_for_rows(L, a, a.grid_share));
    cfg.blockDim = dim3((unsigned)L.threads + side.chunk_units);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, a, side);
}

// The wide vector kernel with or without the coordinate table; the table variants exist for
// the cases launch_one uses them in.
template <int W, int NU, bool MESH, bool COMPACT>
cudaError_t launch_rows_wide(bool tab, const LaunchPlan &L, const LaunchDev &a, cudaStream_t stream, bool dependent)
{
    if constexpr (!MESH && (COMPACT || NU <= 2)) {
        if (tab) return launch_wide(iso_gather_rows_wide<W, kWideDepth, NU, MESH, COMPACT, true>, L, a, stream, dependent);
    }
    return launch_wide(iso_gather_rows_wide<W, kWideDepth, NU, MESH, COMPACT, false>, L, a, stream, dependent);
}

int launch_one(const Request &r, const LaunchPlan &L, cudaStream_t stream, bool dependent, long long row_lo = 0,
               long long row_hi = -1, long long inter_row_base = 0, int grid_share = 1)
{
    if (L.grid == 0 || L.units_per_proc == 0) return ISO_SUCCESS;
    LaunchDev a = make_launch_args(r, L);
    a.grid_share = grid_share;
    if (row_hi >= 0) {
        a.row_lo = row_lo;
        a.row_hi = row_hi;
        if (row_hi <= row_lo) return ISO_SUCCESS;
    }
    // bulk kernel on a range of rows (a slab): its tiles were sized for the whole torus; keep at
    // least two CTAs per SM busy on the range (a smaller tile needs less of the planned shared memory)
    if (L.kernel == KERNEL_BULK && a.row_hi - a.row_lo < a.P) {
        const long long per = std::max<long long>(1, (a.row_hi - a.row_lo) / ((long long)r.sm_count * 2));
        a.tile_procs = (int)std::max<long long>(1, std::min<long long>(L.tile_procs, per));
    }
    // slab-serial execution: the intermediate buffer only holds one slab, addressed from
    // the slab's first row
    if (inter_row_base && a.buf[ISO_BUF_INTER]) a.buf[ISO_BUF_INTER] -= inter_row_base * r.inter_stride;
    cudaError_t e;
    if (L.kernel == KERNEL_BULK) {
        e = launch_kernel(iso_gather_bulk, L, a, stream, dependent);
    } else if (L.kernel == KERNEL_FAN) {
        e = launch_wide(iso_fan_rows<kWideDepth>, L, a, stream, dependent);
    } else if (!L.side.empty()) {
        // mixed-width launch with a bulk side: vector warps + one bulk warp per CTA
        LaunchDev sd = make_launch_args(r, L.side[0]);
        sd.row_lo = a.row_lo;
        sd.row_hi = a.row_hi;
        if (inter_row_base && sd.buf[ISO_BUF_INTER]) sd.buf[ISO_BUF_INTER] -= inter_row_base * r.inter_stride;
        const long long groups = (a.row_hi - a.row_lo + L.rows_per_pass - 1) / L.rows_per_pass;
        const long long grid = grid_for_rows(L, a, a.grid_share);
        bool tab = false;
        if (L.n_used > 0 && L.n_used <= 2 && r.knobs.coord_table) {
            a.tab_iters = (uint32_t)((groups + grid - 1) / grid);
            a.tab_stride = 4;
            tab = L.smem + table_bytes(a) + 128 + L.side[0].smem <= (size_t)kMaxDynamicSmem;
            if (!tab) a.tab_iters = 0;
        }
        sd.chunk_units = (uint32_t)L.side[0].threads;
        sd.side_offset = (uint32_t)((L.smem + table_bytes(a) + 127) / 128 * 128);
        const size_t smem = sd.side_offset + L.side[0].smem;
        e = L.n_used == 0   ? launch_hybrid(iso_gather_rows_hybrid<kHybridDepth, 0, false>, L, a, sd, smem, stream, dependent)
            : L.n_used == 1 ? (tab ? launch_hybrid(iso_gather_rows_hybrid<kHybridDepth, 1, true>, L, a, sd, smem, stream, dependent)
                                   : launch_hybrid(iso_gather_rows_hybrid<kHybridDepth, 1, false>, L, a, sd, smem, stream, dependent))
            : L.n_used == 2 ? (tab ? launch_hybrid(iso_gather_rows_hybrid<kHybridDepth, 2, true>, L, a, sd, smem, stream, dependent)
                                   : launch_hybrid(iso_gather_rows_hybrid<kHybridDepth, 2, false>, L, a, sd, smem, stream, dependent))
                            : launch_hybrid(iso_gather_rows_hybrid<kHybridDepth, 3, false>, L, a, sd, smem, stream, dependent);
    } else if (L.width > 0 && L.width < 4) {
        e = L.width == 2 ? launch_kernel(iso_gather_rows_reg<2, 4>, L, a, stream, dependent)
                         : launch_kernel(iso_gather_rows_reg<1, 4>, L, a, stream, dependent);
    } else {
        // kernels specialised on the number of shifted dimensions; meshes take the general one
        // (with compact unit descriptors: on the dimensions one unit is shifted along)
        const int count = L.compact ? L.max_nnz : L.n_used;
        const int nu = count <= 3 ? count : ISO_MAX_DIMS;
        // wide CTAs: a table of the coordinates of the rows a CTA visits, if it fits behind the ring
        bool tab = false;
        // (measured: +2 to +5 % on the phases of the combining schedules, which shift along one
        // dimension, and on the compact last phase of 16-byte blocks; the one-pass direct
        // schedules, three or more wrap tests per row, are bound by the latency of their
        // scattered loads and gain nothing, so they keep the divisions)
        if ((L.width == 16 || L.width == 0) && L.threads > 256 && L.n_used > 0 && r.knobs.coord_table &&
            (L.compact || nu <= 2) && !a.mesh_mask) {
            const long long groups = (a.row_hi - a.row_lo + L.rows_per_pass - 1) / L.rows_per_pass;
            const long long grid = grid_for_rows(L, a, a.grid_share) / std::max(1, L.col_split);  // CTAs that share the rows
            a.tab_iters = (uint32_t)((groups + grid - 1) / grid);
            a.tab_stride = L.n_used <= 4 ? 4 : 8;
            tab = L.smem + table_bytes(a) <= (size_t)kMaxDynamicSmem;
            if (!tab) a.tab_iters = 0;
        }
#define ISO_ROWS(W, NU, MESH, COMPACT)                                                                          \
    e = ((W == 16 || W == 0) && L.threads > 256)                                                                \
            ? launch_rows_wide<(W == 0 ? 0 : 16), NU, MESH, COMPACT>(tab, L, a, stream, dependent)             \
            : launch_kernel(iso_gather_rows<W, kVecDepth, NU, MESH, COMPACT>, L, a, stream, dependent)
#define ISO_ROWS_W(W)                                                            \
    do {                                                                         \
        if (a.mesh_mask) ISO_ROWS(W, ISO_MAX_DIMS, true, false);                 \
        else if (L.compact && nu == 1) ISO_ROWS(W, 1, false, true);              \
        else if (L.compact && nu == 2) ISO_ROWS(W, 2, false, true);              \
        else if (L.compact && nu == 3) ISO_ROWS(W, 3, false, true);              \
        else if (L.compact) ISO_ROWS(W, ISO_MAX_DIMS, false, true);              \
        else if (nu == 0) ISO_ROWS(W, 0, false, false);                          \
        else if (nu == 1) ISO_ROWS(W, 1, false, false);                          \
        else if (nu == 2) ISO_ROWS(W, 2, false, false);                          \
        else if (nu == 3) ISO_ROWS(W, 3, false, false);                          \
        else ISO_ROWS(W, ISO_MAX_DIMS, false, false);                            \
    } while (0)
        if (L.width == 0) ISO_ROWS_W(0);
        else if (L.width == 16) ISO_ROWS_W(16);
        else if (L.width == 8) ISO_ROWS_W(8);
        else ISO_ROWS_W(4);
#undef ISO_ROWS_W
#undef ISO_ROWS
    }
    ISO_CUDA(e);
    return ISO_SUCCESS;
}

// Slabs of the leading dimension for the pipelined host-buffer path.
struct SlabPlan {
    long long row_lo, row_hi;
    int last_needed;  // index of the last slab whose send buffers this slab's schedule reads
    unsigned long long needs;  // bit j: the slab's schedule reads send buffers of slab j (valid up to 64 slabs)
};

// Fills `slabs` when the schedule can run slab by slab: every part that shifts along
// dimension 0 must read the send buffer (everything else then stays inside a plane of
// dimension 0), all dimensions periodic, and at least four planes.  Leaves it empty otherwise.
void plan_slabs(const Request &r, std::vector<SlabPlan> &slabs, int want = 0)
{
    const Comm &c = *r.comm;
    slabs.clear();
    const int p0 = c.dims[0];
    if (c.d < 2 || p0 < 4 || r.launches.empty()) return;
    for (int j = 0; j < c.d; ++j)
        if (!c.periodic[j]) return;
    std::vector<int> shifts;  // distinct shifts along dimension 0 (0 included)
    shifts.push_back(0);
    for (const LaunchPlan &L : r.launches)
        if (L.kernel == KERNEL_FAN) return;  // a sender-side launch writes outside the rows it is given
    for (const LaunchPlan &L : r.launches)
        for (const LoweredPart &lp : L.parts) {
            const int s0 = lp.p.shift[0];
            if (s0 == 0) continue;
            if (lp.p.src_buf != ISO_BUF_SEND) return;
            if (std::find(shifts.begin(), shifts.end(), s0) == shifts.end()) shifts.push_back(s0);
        }
    // default: up to 32 slabs.  The last slabs to arrive (a slab and the neighbours it reads
    // from) can only run and travel back after the final upload, so the tail of the pipeline
    // is about three slabs long: a quarter of the transfer time with 8 slabs, a tenth with 32.
    int n = std::min(p0, 32);
    if (want > 0) {
        n = std::min(p0, want);
    } else if (r.knobs.host_slabs >= 0) {
        const int v = r.knobs.host_slabs;
        if (v <= 1) return;
        n = std::min(p0, v);
    }
    const long long plane = c.rank_stride[0];
    std::vector<int> slab_of(p0);
    for (int k = 0; k < n; ++k) {
        const int a = (int)((long long)p0 * k / n), b = (int)((long long)p0 * (k + 1) / n);
        for (int x = a; x < b; ++x) slab_of[x] = k;
        slabs.push_back(SlabPlan{a * plane, b * plane, k, 0ULL});
    }
    for (int x = 0; x < p0; ++x)
        for (int s0 : shifts) {
            const int src = ((x - s0) % p0 + p0) % p0;
            slabs[slab_of[x]].last_needed = std::max(slabs[slab_of[x]].last_needed, slab_of[src]);
            if (slab_of[src] < 64) slabs[slab_of[x]].needs |= 1ULL << slab_of[src];
        }
}

// Whether `p` is page-locked host memory (only such copies are recorded into a graph).
bool page_locked(const void *p)
{
    cudaPointerAttributes at{};
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return false;
    }
    return at.type == cudaMemoryTypeHost;
}

// Streams and events of the pipelined host-buffer path: two streams per direction (a copy
// costs about 20 microseconds before its first byte moves; with the copies of a direction
// dealt to two streams the next copy's set-up runs under the current copy's transfer).
int prepare_host_pipeline(Request &r, size_t S)
{
    while (r.host_streams.size() < 4) {
        cudaStream_t st;
        ISO_CUDA(cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking));
        r.host_streams.push_back(st);
    }
    while (r.slab_events.size() < 2 * S + 4) {
        cudaEvent_t e;
        ISO_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        r.slab_events.push_back(e);
    }
    // timing events for Iso_request_get_host_transfer_ms: begin and end of the uploads, of the
    // downloads and of the whole call
    while (r.host_timing.size() < 6) {
        cudaEvent_t e;
        ISO_CUDA(cudaEventCreate(&e));
        r.host_timing.push_back(e);
    }
    return ISO_SUCCESS;
}

// Enqueues one pipelined host-buffer start.  Only blocks read from the send buffer cross
// slabs, so a slab's whole schedule can run as soon as the send buffers of the slabs it reads
// have arrived, and its receive buffers can travel back while later slabs are still on their
// way in.  Five streams: uploads alternate between two, kernels run on `stream`, downloads
// alternate between two more, so that both directions of the link are busy at the same time
// and no copy waits behind a kernel.  With `capturing` the calls are being recorded into a
// graph (`stream` is the capture's origin): the timing events then become external event nodes.
int enqueue_host_pipeline(Request &r, const std::vector<SlabPlan> &slabs, const unsigned char *hs, unsigned char *hr,
                          cudaStream_t stream, bool capturing)
{
    const Comm &c = *r.comm;
    const size_t S = slabs.size();
    cudaStream_t up[2] = {static_cast<cudaStream_t>(r.host_streams[0]), static_cast<cudaStream_t>(r.host_streams[1])};
    cudaStream_t down[2] = {static_cast<cudaStream_t>(r.host_streams[2]), static_cast<cudaStream_t>(r.host_streams[3])};
    auto stamp = [&](void *event, cudaStream_t on) -> cudaError_t {
        return cudaEventRecordWithFlags(static_cast<cudaEvent_t>(event), on, capturing ? cudaEventRecordExternal : cudaEventRecordDefault);
    };
    auto event = [&](size_t k) { return static_cast<cudaEvent_t>(r.slab_events[k]); };
    // copies of this call must not overtake earlier work on the caller's stream
    cudaEvent_t fence = event(2 * S);
    ISO_CUDA(cudaEventRecord(fence, stream));
    for (int k = 0; k < 2; ++k) {
        ISO_CUDA(cudaStreamWaitEvent(up[k], fence, 0));
        ISO_CUDA(cudaStreamWaitEvent(down[k], fence, 0));
    }
    ISO_CUDA(stamp(r.host_timing[4], stream));
    ISO_CUDA(stamp(r.host_timing[0], up[0]));
    size_t downloads = 0;
    const bool use_pdl = !r.knobs.no_pdl;
    // Upload order: the last slab first, then 0, 1, ...: on a torus slab 0 reads the last slab,
    // so in natural order it (and its download) would have to wait for the very last upload.
    std::vector<size_t> order(S), pos(S);
    for (size_t i = 0; i < S; ++i) order[i] = S <= 64 ? (i + S - 1) % S : i;
    for (size_t i = 0; i < S; ++i) pos[order[i]] = i;
    std::vector<size_t> ready_at(S, 0);  // position in the upload order after which a slab can run
    for (size_t k = 0; k < S; ++k) {
        if (S <= 64) {
            for (size_t j = 0; j < S; ++j)
                if (slabs[k].needs >> j & 1ULL) ready_at[k] = std::max(ready_at[k], pos[j]);
            ready_at[k] = std::max(ready_at[k], pos[k]);
        } else {
            ready_at[k] = (size_t)std::max(slabs[k].last_needed, (int)k);
        }
    }
    std::vector<char> done(S, 0);
    for (size_t upi = 0; upi < S; ++upi) {
        const SlabPlan &u = slabs[order[upi]];
        const size_t off = (size_t)(u.row_lo * r.send_stride), n = (size_t)((u.row_hi - u.row_lo) * r.send_stride);
        if (n) ISO_CUDA(cudaMemcpyAsync(const_cast<unsigned char *>(r.send) + off, hs + off, n, cudaMemcpyHostToDevice, up[upi & 1]));
        ISO_CUDA(cudaEventRecord(event(S + upi), up[upi & 1]));
        // every slab whose last needed upload this was: it follows this upload and the one
        // before it, which is the latest on the other upload stream
        for (size_t k = 0; k < S; ++k) {
            if (done[k] || ready_at[k] > upi) continue;
            const SlabPlan &w = slabs[k];
            ISO_CUDA(cudaStreamWaitEvent(stream, event(S + upi), 0));
            if (upi > 0) ISO_CUDA(cudaStreamWaitEvent(stream, event(S + upi - 1), 0));
            for (const LaunchPlan &L : r.launches) {
                int rc = launch_one(r, L, stream, use_pdl, w.row_lo, w.row_hi, r.inter_rows < c.P ? w.row_lo : 0);
                if (rc != ISO_SUCCESS) return rc;
            }
            ISO_CUDA(cudaEventRecord(event(k), stream));
            cudaStream_t dn = down[downloads & 1];
            ISO_CUDA(cudaStreamWaitEvent(dn, event(k), 0));
            if (downloads == 0) ISO_CUDA(stamp(r.host_timing[2], dn));
            ++downloads;
            const size_t roff = (size_t)(w.row_lo * r.recv_stride), rn = (size_t)((w.row_hi - w.row_lo) * r.recv_stride);
            if (rn) ISO_CUDA(cudaMemcpyAsync(hr + roff, r.recv + roff, rn, cudaMemcpyDeviceToHost, dn));
            done[k] = 1;
        }
    }
    // join: the caller's stream is complete only when every copy stream is (a capture must
    // end with every forked stream joined); the time stamps follow the joins
    ISO_CUDA(cudaEventRecord(event(2 * S + 1), up[1]));
    ISO_CUDA(cudaStreamWaitEvent(up[0], event(2 * S + 1), 0));
    ISO_CUDA(stamp(r.host_timing[1], up[0]));
    ISO_CUDA(cudaEventRecord(event(2 * S + 2), down[1]));
    ISO_CUDA(cudaStreamWaitEvent(down[0], event(2 * S + 2), 0));
    ISO_CUDA(stamp(r.host_timing[3], down[0]));
    ISO_CUDA(cudaEventRecord(fence, down[0]));
    ISO_CUDA(cudaStreamWaitEvent(stream, fence, 0));
    ISO_CUDA(cudaEventRecord(event(2 * S + 3), up[0]));
    ISO_CUDA(cudaStreamWaitEvent(stream, event(2 * S + 3), 0));
    ISO_CUDA(stamp(r.host_timing[5], stream));
    return ISO_SUCCESS;
}

// No exception may cross the C boundary: allocation failures become ISO_ERR_NOMEM.
template <typename F>
int guarded(F &&f) noexcept
{
    try {
        return f();
    } catch (const std::bad_alloc &) {
        return ISO_ERR_NOMEM;
    } catch (...) {
        return ISO_ERR_STATE;
    }
}

// Decides whether Iso_Start runs slab after slab (and how many slabs), and how many rows the
// intermediate buffer has to hold.  Automatic rule: all-to-all schedules of vector launches
// only (the bulk kernel and the allgather measured slower in slabs) with enough work per
// slab; measured gains 10-16 % on the 256^2 torus with 64-byte blocks (2 slabs) and on the
// 63-, 80- and 342-neighbour workloads (2 to 16 slabs), none on the 32^3 torus (1 slab).
void choose_slab_plan(Request &r)
{
    const Comm &c = *r.comm;
    r.slab_plan.clear();
    r.inter_rows = c.P;
    r.chains = 1;
    r.use_graph = !r.persistent && r.graph_request;
    if (r.knobs.graph >= 0) r.use_graph = !r.persistent && r.knobs.graph != 0;
    if (r.wave_ok) {
        // pipelined one-launch execution: its own slabs; from three slabs on the
        // intermediate buffer holds two of them
        r.use_graph = false;
        if (r.wave_request >= 2 && r.inter_stride > 0) {
            std::vector<SlabPlan> slabs;
            plan_slabs(r, slabs, r.wave_request);
            long long rows = 0;
            if (slabs.size() >= 2)
                for (const SlabPlan &w : slabs) {
                    r.slab_plan.push_back({w.row_lo, w.row_hi});
                    rows = std::max(rows, w.row_hi - w.row_lo);
                }
            if (r.slab_plan.size() >= 3) r.inter_rows = 2 * rows;
        }
        return;
    }
    if (r.persistent || r.inter_stride == 0) return;
    int want = r.slab_request;
    if (r.knobs.slabs >= 0) want = r.knobs.slabs;
    if (want == 0) {
        // automatic: all-to-all schedules made of vector launches only.  What one launch of a slab
        // writes the next one reads back, so both should sit in the L2 (126 MB) together: the
        // fewest slabs (a power of two) that bring a launch's written bytes under 52 MB, as long
        // as every CTA still gets half a dozen rows.  Measured optimum and this rule's choice on
        // nine all-to-all workloads (64-byte blocks unless stated): 32^3 Moore r=1 1 and 1, 256^2
        // Moore r=2 2 and 2, 8^5 16-byte blocks 2 and 2, positive octant 2 and 2, stencil-shaped
        // sizes 4 and 2 (5 % apart), 16^4 Moore r=1 8 and 8, Moore r=3 16 and 16, shells 32 and 32,
        // irregular 64x64x32 64 and 32 (1.5 % apart).
        if (r.kind == ISO_KIND_ALLGATHER) return;
        long long rows_per_pass = 1;
        for (const LaunchPlan &L : r.launches) {
            if (L.kernel != KERNEL_VEC) return;
            rows_per_pass = std::max<long long>(rows_per_pass, L.rows_hint > 0 ? (long long)L.rows_hint : (long long)L.grid * L.rows_per_pass);
        }
        const double written = (double)r.stats.bytes_moved / 2.0 / (double)std::max<size_t>(1, r.launches.size());
        int target = 1;
        while (target < kMaxOwnSlabs && written / target > kSlabLaunchBytes) target *= 2;
        want = 1;
        while (want < target && c.P / (want * 2) >= 6 * rows_per_pass) want *= 2;
    }
    int chains = std::max(1, r.chains_request);
    if (r.knobs.chains >= 0) chains = std::max(1, std::min(8, r.knobs.chains));
    if (chains > 1) want = std::max(want, chains) / chains * chains;
    if (want < 2) return;
    std::vector<SlabPlan> slabs;
    plan_slabs(r, slabs, want);
    if (slabs.size() < 2) return;
    long long rows = 0;
    for (const SlabPlan &w : slabs) {
        r.slab_plan.push_back({w.row_lo, w.row_hi});
        rows = std::max(rows, w.row_hi - w.row_lo);
    }
    if (chains > 1 && slabs.size() % chains == 0) {
        // slabs side by side: every chain has its own one-slab part of the intermediate buffer
        r.chains = chains;
        r.use_graph = true;
        rows *= chains;
    }
    // a start of very many launches is replayed from a graph unless the environment says otherwise
    // (4 KB blocks on the 256x256 torus, 256 launches per start: 3.16 -> 3.10 ms; at 96 launches
    // per start and below replay measured no gain)
    if (r.knobs.graph < 0 && r.slab_plan.size() * r.launches.size() >= 128) r.use_graph = true;
    // the pipelined host-buffer path cuts dimension 0 into slabs of its own (plan_slabs)
    std::vector<SlabPlan> host;
    plan_slabs(r, host);
    for (const SlabPlan &w : host) rows = std::max(rows, w.row_hi - w.row_lo);
    r.inter_rows = rows;
}

int check_handle(Iso_request request)
{
    return request && request->comm ? ISO_SUCCESS : ISO_ERR_ARG;
}

// Captures the launches of one Iso_Start into a graph.  With r.chains > 1 the slabs are
// dealt to that many chains, which run side by side: chain k takes the slabs k, k + chains,
// ..., a 1/chains share of the CTA slots and its own part of the intermediate buffer, so
// that the ramp and the drain of one chain's kernels are covered by the other chains.
int build_graph(Request &r, bool use_pdl)
{
    const int n = std::max(1, r.chains);
    std::vector<cudaStream_t> st(n, nullptr);
    std::vector<cudaEvent_t> ev(n, nullptr);
    cudaError_t e = cudaSuccess;
    for (int k = 0; k < n && e == cudaSuccess; ++k) {
        e = cudaStreamCreateWithFlags(&st[k], cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ev[k], cudaEventDisableTiming);
    }
    cudaGraph_t graph = nullptr;
    int rc = ISO_SUCCESS;
    bool capturing = false;
    if (e == cudaSuccess) e = cudaStreamBeginCapture(st[0], cudaStreamCaptureModeThreadLocal);
    if (e == cudaSuccess) {
        capturing = true;
        e = cudaEventRecord(ev[0], st[0]);
        for (int k = 1; k < n && e == cudaSuccess; ++k) e = cudaStreamWaitEvent(st[k], ev[0], 0);
    }
    if (e == cudaSuccess) {
        if (r.slab_plan.size() > 1) {
            long long slab_rows = 0;
            for (const auto &w : r.slab_plan) slab_rows = std::max(slab_rows, w.second - w.first);
            for (size_t i = 0; i < r.slab_plan.size() && rc == ISO_SUCCESS; ++i) {
                const int k = (int)(i % (size_t)n);
                const auto &w = r.slab_plan[i];
                bool first = i < (size_t)n;  // nothing of this chain precedes it in its stream
                for (const LaunchPlan &L : r.launches) {
                    rc = launch_one(r, L, st[k], use_pdl && !first, w.first, w.second, w.first - (long long)k * slab_rows, n);
                    first = false;
                    if (rc != ISO_SUCCESS) break;
                }
            }
        } else {
            bool first = true;
            for (const LaunchPlan &L : r.launches) {
                rc = launch_one(r, L, st[0], use_pdl && !first);
                first = false;
                if (rc != ISO_SUCCESS) break;
            }
        }
        for (int k = 1; k < n && e == cudaSuccess; ++k) {
            e = cudaEventRecord(ev[k], st[k]);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(st[0], ev[k], 0);
        }
    }
    if (capturing) {
        cudaError_t e2 = cudaStreamEndCapture(st[0], &graph);
        if (e == cudaSuccess) e = e2;
    }
    cudaGraphExec_t exec = nullptr;
    if (e == cudaSuccess && rc == ISO_SUCCESS) e = cudaGraphInstantiate(&exec, graph, 0);
    if (graph) cudaGraphDestroy(graph);
    for (int k = 0; k < n; ++k) {
        if (ev[k]) cudaEventDestroy(ev[k]);
        if (st[k]) cudaStreamDestroy(st[k]);
    }
    if (rc != ISO_SUCCESS) return rc;
    if (e != cudaSuccess) return cuda_fail(e);
    r.graph_exec = exec;
    return ISO_SUCCESS;
}

}  // namespace

extern "C" {

int Iso_neighborhood_create(int d, const int dims[], int s, const int relative_coordinates[], Iso_comm *isocomm)
{
    return guarded([&]() -> int {
    if (!isocomm || !dims || s < 0 || (s > 0 && !relative_coordinates)) return ISO_ERR_ARG;
    if (d < 1 || d > ISO_MAX_DIMS) return ISO_ERR_DIMS;
    int64_t P = 1;
    for (int j = 0; j < d; ++j) {
        if (dims[j] < 1) return ISO_ERR_DIMS;
        if (P > (int64_t)0x7fffffff / dims[j]) return ISO_ERR_DIMS;  // ranks are kept below 2^31
        P *= dims[j];
    }
    Iso_comm_s *c = new (std::nothrow) Iso_comm_s();
    if (!c) return ISO_ERR_NOMEM;
    c->d = d;
    c->s = s;
    c->P = P;
    int64_t stride = 1;
    for (int j = d - 1; j >= 0; --j) {
        c->dims[j] = dims[j];
        c->periodic[j] = 1;
        c->rank_stride[j] = stride;
        stride *= dims[j];
    }
    try {
        c->coords.assign(relative_coordinates, relative_coordinates + (size_t)s * d);
    } catch (...) {
        delete c;
        return ISO_ERR_NOMEM;
    }
    *isocomm = c;
    return ISO_SUCCESS;
    });
}

int Iso_comm_set_periodic(Iso_comm isocomm, const int periodic[])
{
    if (!isocomm || !periodic) return ISO_ERR_ARG;
    for (int j = 0; j < isocomm->d; ++j) isocomm->periodic[j] = periodic[j] ? 1 : 0;
    return ISO_SUCCESS;
}

int Iso_comm_free(Iso_comm *isocomm)
{
    if (!isocomm || !*isocomm) return ISO_ERR_ARG;
    comm_unref(*isocomm);
    *isocomm = nullptr;
    return ISO_SUCCESS;
}

int Iso_neighbor_alltoall_init(const void *sendbuf, int sendcount, Iso_datatype sendtype, void *recvbuf,
                               int recvcount, Iso_datatype recvtype, Iso_comm isocomm, Iso_request *request)
{
    return guarded([&]() -> int {
    if (!isocomm || !request || sendcount < 0 || recvcount < 0 || sendtype < 1 || recvtype < 1) return ISO_ERR_ARG;
    if ((sendbuf == nullptr) != (recvbuf == nullptr)) return ISO_ERR_ARG;
    const int64_t m = (int64_t)sendcount * sendtype;
    if (m != (int64_t)recvcount * recvtype) return ISO_ERR_COUNT;
    Iso_request_s *r = new_request(isocomm, ISO_KIND_ALLTOALL, sendbuf, recvbuf);
    if (!r) return ISO_ERR_NOMEM;
    for (int i = 0; i < r->s; ++i) {
        r->len[i] = m;
        r->sdispl[i] = r->rdispl[i] = (int64_t)i * m;
    }
    r->send_stride = r->recv_stride = (int64_t)r->s * m;
    return finish_init(r, request);
    });
}

int Iso_neighbor_allgather_init(const void *sendbuf, int sendcount, Iso_datatype sendtype, void *recvbuf,
                                int recvcount, Iso_datatype recvtype, Iso_comm isocomm, Iso_request *request)
{
    return guarded([&]() -> int {
    if (!isocomm || !request || sendcount < 0 || recvcount < 0 || sendtype < 1 || recvtype < 1) return ISO_ERR_ARG;
    if ((sendbuf == nullptr) != (recvbuf == nullptr)) return ISO_ERR_ARG;
    const int64_t m = (int64_t)sendcount * sendtype;
    if (m != (int64_t)recvcount * recvtype) return ISO_ERR_COUNT;
    Iso_request_s *r = new_request(isocomm, ISO_KIND_ALLGATHER, sendbuf, recvbuf);
    if (!r) return ISO_ERR_NOMEM;
    for (int i = 0; i < r->s; ++i) {
        r->len[i] = m;
        r->sdispl[i] = 0;
        r->rdispl[i] = (int64_t)i * m;
    }
    r->send_stride = m;
    r->recv_stride = (int64_t)r->s * m;
    return finish_init(r, request);
    });
}

int Iso_neighbor_alltoallv_init(const void *sendbuf, const int sendcounts[], const int64_t senddispls[],
                                Iso_datatype sendtype, void *recvbuf, const int recvcounts[],
                                const int64_t recvdispls[], Iso_datatype recvtype, Iso_comm isocomm,
                                Iso_request *request)
{
    return guarded([&]() -> int {
    if (!isocomm || !request || sendtype < 1 || recvtype < 1) return ISO_ERR_ARG;
    if (isocomm->s > 0 && (!sendcounts || !senddispls || !recvcounts || !recvdispls)) return ISO_ERR_ARG;
    if ((sendbuf == nullptr) != (recvbuf == nullptr)) return ISO_ERR_ARG;
    for (int i = 0; i < isocomm->s; ++i) {
        if (sendcounts[i] < 0 || recvcounts[i] < 0 || senddispls[i] < 0 || recvdispls[i] < 0) return ISO_ERR_ARG;
        if ((int64_t)sendcounts[i] * sendtype != (int64_t)recvcounts[i] * recvtype) return ISO_ERR_COUNT;
    }
    Iso_request_s *r = new_request(isocomm, ISO_KIND_ALLTOALLV, sendbuf, recvbuf);
    if (!r) return ISO_ERR_NOMEM;
    int64_t se = 0, re = 0;
    for (int i = 0; i < r->s; ++i) {
        r->len[i] = (int64_t)sendcounts[i] * sendtype;
        r->sdispl[i] = senddispls[i];
        r->rdispl[i] = recvdispls[i];
        se = std::max(se, senddispls[i] + r->len[i]);
        re = std::max(re, recvdispls[i] + r->len[i]);
    }
    r->send_stride = round_up16(se);
    r->recv_stride = round_up16(re);
    return finish_init(r, request);
    });
}

int Iso_neighbor_allgatherv_init(const void *sendbuf, int sendcount, Iso_datatype sendtype, void *recvbuf,
                                 const int recvcounts[], const int64_t recvdispls[], Iso_datatype recvtype,
                                 Iso_comm isocomm, Iso_request *request)
{
    return guarded([&]() -> int {
    if (!isocomm || !request || sendcount < 0 || sendtype < 1 || recvtype < 1) return ISO_ERR_ARG;
    if (isocomm->s > 0 && (!recvcounts || !recvdispls)) return ISO_ERR_ARG;
    if ((sendbuf == nullptr) != (recvbuf == nullptr)) return ISO_ERR_ARG;
    const int64_t m = (int64_t)sendcount * sendtype;
    for (int i = 0; i < isocomm->s; ++i) {
        if (recvcounts[i] < 0 || recvdispls[i] < 0) return ISO_ERR_ARG;
        if ((int64_t)recvcounts[i] * recvtype != m) return ISO_ERR_COUNT;
    }
    Iso_request_s *r = new_request(isocomm, ISO_KIND_ALLGATHER, sendbuf, recvbuf);
    if (!r) return ISO_ERR_NOMEM;
    int64_t re = 0;
    for (int i = 0; i < r->s; ++i) {
        r->len[i] = m;
        r->sdispl[i] = 0;
        r->rdispl[i] = recvdispls[i];
        re = std::max(re, recvdispls[i] + m);
    }
    r->send_stride = round_up16(m);
    r->recv_stride = round_up16(re);
    return finish_init(r, request);
    });
}

int Iso_request_set_algorithm(Iso_request request, int alg, int fusion_level)
{
    return guarded([&]() -> int {
    if (check_handle(request)) return ISO_ERR_ARG;
    if (alg != ISO_ALG_COMBINING && alg != ISO_ALG_DIRECT && alg != ISO_ALG_TORUS) return ISO_ERR_ARG;
    if (fusion_level < 0) return ISO_ERR_ARG;
    if (request->started) {
        int rc = Iso_wait(request);
        if (rc != ISO_SUCCESS) return rc;
    }
    const int old_alg = request->alg, old_fusion = request->fusion;
    request->alg = alg;
    request->fusion = fusion_level;
    int rc = build_schedule(*request);
    if (rc == ISO_SUCCESS)
        rc = lower_schedule(*request, (uintptr_t)request->send, (uintptr_t)request->recv, (uintptr_t)request->d_inter);
    if (rc != ISO_SUCCESS) {
        request->alg = old_alg;
        request->fusion = old_fusion;
        build_schedule(*request);
        lower_schedule(*request, (uintptr_t)request->send, (uintptr_t)request->recv, (uintptr_t)request->d_inter);
    }
    request->dirty = true;
    return rc;
    });
}

int Iso_request_set_layout(Iso_request request, int layout)
{
    return guarded([&]() -> int {
    if (check_handle(request) || (layout != ISO_LAYOUT_PACKED && layout != ISO_LAYOUT_ALTERNATING)) return ISO_ERR_ARG;
    request->layout = layout;
    if (request->alg != ISO_ALG_COMBINING) return ISO_SUCCESS;  // takes effect with the next combining schedule
    return Iso_request_set_algorithm(request, request->alg, request->fusion);
    });
}

int Iso_request_set_single_launch(Iso_request request, int enable)
{
    return guarded([&]() -> int {
    if (check_handle(request)) return ISO_ERR_ARG;
    if (request->started) {
        int rc = Iso_wait(request);
        if (rc != ISO_SUCCESS) return rc;
    }
    request->persistent = enable != 0;
    request->dirty = true;
    return ISO_SUCCESS;
    });
}

int Iso_request_set_pipeline(Iso_request request, int slabs)
{
    return guarded([&]() -> int {
    if (check_handle(request) || slabs < 0) return ISO_ERR_ARG;
    if (request->started) {
        int rc = Iso_wait(request);
        if (rc != ISO_SUCCESS) return rc;
    }
    request->wave_request = slabs;
    request->dirty = true;
    return ISO_SUCCESS;
    });
}

int Iso_request_set_slabs(Iso_request request, int slabs)
{
    return guarded([&]() -> int {
    if (check_handle(request) || slabs < 0) return ISO_ERR_ARG;
    if (request->started) {
        int rc = Iso_wait(request);
        if (rc != ISO_SUCCESS) return rc;
    }
    request->slab_request = slabs;
    request->dirty = true;
    // (which kernel moves the longer parts depends on who chooses the slabs)
    return lower_schedule(*request, (uintptr_t)request->send, (uintptr_t)request->recv, (uintptr_t)request->d_inter);
    });
}

int Iso_request_set_chains(Iso_request request, int chains)
{
    return guarded([&]() -> int {
    if (check_handle(request) || chains < 1 || chains > 8) return ISO_ERR_ARG;
    if (request->started) {
        int rc = Iso_wait(request);
        if (rc != ISO_SUCCESS) return rc;
    }
    request->chains_request = chains;
    request->dirty = true;
    return ISO_SUCCESS;
    });
}

int Iso_request_set_graph(Iso_request request, int enable)
{
    return guarded([&]() -> int {
    if (check_handle(request)) return ISO_ERR_ARG;
    if (request->started) {
        int rc = Iso_wait(request);
        if (rc != ISO_SUCCESS) return rc;
    }
    request->graph_request = enable != 0;
    request->dirty = true;
    return ISO_SUCCESS;
    });
}

int Iso_request_get_execution(Iso_request request, int *slabs, int *chains, int *graph)
{
    if (check_handle(request)) return ISO_ERR_ARG;
    const Request &r = *request;
    if (slabs) *slabs = r.dirty ? r.slab_request : (int)std::max<size_t>(1, r.slab_plan.size());
    if (chains) *chains = r.dirty ? r.chains_request : r.chains;
    if (graph) *graph = r.dirty ? (r.graph_request ? 1 : 0) : (r.use_graph ? 1 : 0);
    return ISO_SUCCESS;
}

int Iso_request_tune(Iso_request request, void *cuda_stream, int flags)
{
    return guarded([&]() -> int {
    if (check_handle(request) || (flags & ~(ISO_TUNE_COLD | ISO_TUNE_SCHEDULE))) return ISO_ERR_ARG;
    const bool cold = (flags & ISO_TUNE_COLD) != 0;
    Request &r = *request;
    if (!r.send || !r.recv) return ISO_ERR_STATE;
    if (r.persistent || r.wave_request > 0) return ISO_SUCCESS;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaEvent_t t0 = nullptr, t1 = nullptr;
    ISO_CUDA(cudaEventCreate(&t0));
    if (cudaEventCreate(&t1) != cudaSuccess) {
        cudaEventDestroy(t0);
        return cuda_fail(cudaGetLastError());
    }
    // cold: a scratch buffer of twice the L2 size is overwritten before every timed start
    // (inside the timed span: the same cost for every variant)
    unsigned char *scratch = nullptr;
    size_t scratch_bytes = 0;
    if (cold) {
        int device = 0, l2 = 0;
        cudaGetDevice(&device);
        cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, device);
        scratch_bytes = 2 * (size_t)std::max(l2, 32 << 20);
        if (cudaMalloc((void **)&scratch, scratch_bytes) != cudaSuccess) {
            cudaEventDestroy(t0);
            cudaEventDestroy(t1);
            return cuda_fail(cudaGetLastError());
        }
    }
    const bool log = r.knobs.tune_log;
    // order: visiting order of the allgather's trie (-1: as it was, 0: first dimension first, 1: last first)
    struct Choice { int slabs, chains, graph, alg, fusion, hybrid, order; };
    const Choice before{r.slab_request, r.chains_request, r.graph_request ? 1 : 0, r.alg, r.fusion, r.hybrid ? 1 : 0, -1};
    int order_before[ISO_MAX_DIMS];
    std::copy(r.dim_order, r.dim_order + ISO_MAX_DIMS, order_before);
    int order_now = -1;
    Choice best = before;
    float best_ms = -1.0f;
    int rc = ISO_SUCCESS;
    const int p0 = r.comm->dims[0];
    auto apply = [&](const Choice &c) -> int {
        r.slab_request = c.slabs;
        r.chains_request = c.chains;
        r.graph_request = c.graph != 0;
        r.hybrid = c.hybrid != 0;
        r.dirty = true;
        if (c.order != order_now) {
            int order[ISO_MAX_DIMS];
            for (int k = 0; k < r.comm->d; ++k) order[k] = c.order < 0 ? order_before[k] : (c.order ? r.comm->d - 1 - k : k);
            order_now = c.order;
            r.alg = c.alg;
            r.fusion = c.fusion;
            return Iso_request_set_dimension_order(request, order);  // rebuilds the schedule
        }
        if (c.alg != r.alg || c.fusion != r.fusion) return Iso_request_set_algorithm(request, c.alg, c.fusion);
        return ISO_SUCCESS;
    };
    // the schedules to try: the present one, or - when asked - the message-combining schedule
    // with the hops of 1 and of 2 consecutive dimensions per phase, and the direct schedule
    // (the allgather's message-combining schedule in both visiting orders of the dimensions)
    struct Sched { int first, second, order; };
    std::vector<Sched> schedules(1, Sched{r.alg, r.fusion, -1});
    if (flags & ISO_TUNE_SCHEDULE) {
        const bool orders = r.kind == ISO_KIND_ALLGATHER && r.comm->d >= 2;
        schedules.assign(1, Sched{(int)ISO_ALG_COMBINING, 1, orders ? 0 : -1});
        if (orders) schedules.push_back(Sched{(int)ISO_ALG_COMBINING, 1, 1});
        if (r.comm->d >= 3) schedules.push_back(Sched{(int)ISO_ALG_COMBINING, 2, -1});
        schedules.push_back(Sched{(int)ISO_ALG_DIRECT, 1, -1});
    }
    // time `reps` starts back to back (the collective only reads the send buffers, so
    // repeating it leaves the same result)
    auto measure = [&](int reps, float &ms) -> int {
        for (int k = 0; k < 2; ++k) {
            int e = Iso_Start(request, cuda_stream);
            if (e != ISO_SUCCESS) return e;
        }
        if (cudaEventRecord(t0, stream) != cudaSuccess) return cuda_fail(cudaGetLastError());
        for (int k = 0; k < reps; ++k) {
            if (scratch && cudaMemsetAsync(scratch, k & 0xff, scratch_bytes, stream) != cudaSuccess)
                return cuda_fail(cudaGetLastError());
            int e = Iso_Start(request, cuda_stream);
            if (e != ISO_SUCCESS) return e;
        }
        if (cudaEventRecord(t1, stream) != cudaSuccess) return cuda_fail(cudaGetLastError());
        int e = Iso_wait(request);
        if (e != ISO_SUCCESS) return e;
        if (cudaEventElapsedTime(&ms, t0, t1) != cudaSuccess) return cuda_fail(cudaGetLastError());
        ms /= (float)reps;
        return ISO_SUCCESS;
    };
    // the plan the request came with is the first candidate (with the slab count left to the
    // library it may use kernels that no explicit slab count below selects)
    {
        if (r.started) rc = Iso_wait(request);
        if (rc == ISO_SUCCESS) rc = materialise(r);
        float ms = 0.0f;
        if (rc == ISO_SUCCESS) rc = measure(3, ms);
        if (rc == ISO_SUCCESS) {
            const int reps = (int)std::max(5.0f, std::min(200.0f, 2.0f / std::max(ms, 1e-3f)));
            rc = measure(reps, ms);
        }
        if (rc == ISO_SUCCESS) {
            best_ms = ms;
            if (log) std::fprintf(stderr, "iso tune: as it came: %.4f ms\n", ms);
        }
    }
    for (const auto &sched : schedules)
    for (int hybrid = 0; hybrid <= 1 && rc == ISO_SUCCESS; ++hybrid) {
    if (hybrid) {
        // ragged rows only: does the lowering hand anything to bulk warps?
        r.hybrid = true;
        if (r.started) rc = Iso_wait(request);
        if (rc == ISO_SUCCESS) rc = apply(Choice{1, 1, 0, sched.first, sched.second, 1, sched.order});
        if (rc == ISO_SUCCESS) rc = lower_schedule(r, (uintptr_t)r.send, (uintptr_t)r.recv, (uintptr_t)r.d_inter);
        bool any = false;
        for (const LaunchPlan &L : r.launches) any = any || !L.side.empty();
        if (!any || rc != ISO_SUCCESS) continue;
    }
    std::vector<Choice> tried;
    for (int graph = 0; graph <= 1 && rc == ISO_SUCCESS; ++graph)
        for (int chains = 1; chains <= 4 && rc == ISO_SUCCESS; chains *= 2) {
            if (chains > 1 && !graph) continue;  // chains only exist inside a graph
            for (int slabs = 1; slabs <= 64 && slabs <= std::max(1, p0) && rc == ISO_SUCCESS; slabs *= 2) {
                if (chains > 1 && slabs < chains) continue;
                if (r.started) rc = Iso_wait(request);
                if (rc == ISO_SUCCESS) rc = apply(Choice{slabs, chains, graph, sched.first, sched.second, hybrid, sched.order});
                if (rc == ISO_SUCCESS) rc = materialise(r);
                if (rc != ISO_SUCCESS) break;
                // what the schedule allowed may differ from what was asked for: skip repeats
                const Choice got{(int)std::max<size_t>(1, r.slab_plan.size()), r.chains, r.use_graph ? 1 : 0, r.alg, r.fusion, hybrid, sched.order};
                bool seen = false;
                for (const Choice &c : tried) seen = seen || (c.slabs == got.slabs && c.chains == got.chains && c.graph == got.graph);
                if (seen) continue;
                tried.push_back(got);
                float ms = 0.0f;
                rc = measure(3, ms);  // a first look, then the real measurement scaled to it
                if (rc != ISO_SUCCESS) break;
                const int reps = (int)std::max(5.0f, std::min(200.0f, 2.0f / std::max(ms, 1e-3f)));
                rc = measure(reps, ms);
                if (rc != ISO_SUCCESS) break;
                if (log)
                    std::fprintf(stderr, "iso tune: alg %d fusion %d order %d hybrid %d slabs %d chains %d graph %d: %.4f ms\n", got.alg,
                                 got.fusion, got.order, got.hybrid, got.slabs, got.chains, got.graph, ms);
                // the plainer plans come first; a later one must win by 2 % to replace them
                if (best_ms < 0.0f || ms < 0.98f * best_ms) {
                    best_ms = ms;
                    best = Choice{slabs, chains, graph, sched.first, sched.second, hybrid, sched.order};
                }
            }
        }
    }
    cudaEventDestroy(t0);
    cudaEventDestroy(t1);
    if (scratch) cudaFree(scratch);
    if (r.started) {
        int e = Iso_wait(request);
        if (rc == ISO_SUCCESS) rc = e;
    }
    int e = apply(rc == ISO_SUCCESS ? best : before);
    if (e == ISO_SUCCESS) e = materialise(r);
    return rc != ISO_SUCCESS ? rc : e;
    });
}

int Iso_request_set_hybrid(Iso_request request, int enable)
{
    return guarded([&]() -> int {
    if (check_handle(request)) return ISO_ERR_ARG;
    if (request->started) {
        int rc = Iso_wait(request);
        if (rc != ISO_SUCCESS) return rc;
    }
    request->hybrid = enable != 0;
    int rc = lower_schedule(*request, (uintptr_t)request->send, (uintptr_t)request->recv, (uintptr_t)request->d_inter);
    request->dirty = true;
    return rc;
    });
}

int Iso_request_set_sender_side(Iso_request request, int mode)
{
    return guarded([&]() -> int {
    if (check_handle(request) || mode < 0 || mode > 2) return ISO_ERR_ARG;
    if (request->started) {
        int rc = Iso_wait(request);
        if (rc != ISO_SUCCESS) return rc;
    }
    request->sender_side = mode;
    int rc = lower_schedule(*request, (uintptr_t)request->send, (uintptr_t)request->recv, (uintptr_t)request->d_inter);
    request->dirty = true;
    return rc;
    });
}

int Iso_request_set_dimension_order(Iso_request request, const int order[])
{
    return guarded([&]() -> int {
    if (check_handle(request) || !order) return ISO_ERR_ARG;
    const int d = request->comm->d;
    bool seen[ISO_MAX_DIMS] = {false};
    for (int k = 0; k < d; ++k) {
        if (order[k] < 0 || order[k] >= d || seen[order[k]]) return ISO_ERR_ARG;
        seen[order[k]] = true;
    }
    if (request->started) {
        int rc = Iso_wait(request);
        if (rc != ISO_SUCCESS) return rc;
    }
    int old[ISO_MAX_DIMS];
    std::copy(request->dim_order, request->dim_order + ISO_MAX_DIMS, old);
    std::copy(order, order + d, request->dim_order);
    int rc = build_schedule(*request);
    if (rc == ISO_SUCCESS)
        rc = lower_schedule(*request, (uintptr_t)request->send, (uintptr_t)request->recv, (uintptr_t)request->d_inter);
    if (rc != ISO_SUCCESS) {
        std::copy(old, old + ISO_MAX_DIMS, request->dim_order);
        build_schedule(*request);
        lower_schedule(*request, (uintptr_t)request->send, (uintptr_t)request->recv, (uintptr_t)request->d_inter);
    }
    request->dirty = true;
    return rc;
    });
}

int Iso_request_get_dimension_order(Iso_request request, int order[])
{
    return guarded([&]() -> int {
    if (check_handle(request) || !order) return ISO_ERR_ARG;
    std::copy(request->dim_order, request->dim_order + request->comm->d, order);
    return ISO_SUCCESS;
    });
}

int Iso_request_set_bulk_threshold(Iso_request request, int64_t bytes)
{
    return guarded([&]() -> int {
    if (check_handle(request) || bytes < 0) return ISO_ERR_ARG;
    if (request->started) {
        int rc = Iso_wait(request);
        if (rc != ISO_SUCCESS) return rc;
    }
    request->bulk_threshold_asked = bytes;
    int rc = lower_schedule(*request, (uintptr_t)request->send, (uintptr_t)request->recv, (uintptr_t)request->d_inter);
    request->dirty = true;
    return rc;
    });
}


int Iso_Start(Iso_request request, void *cuda_stream)
{
    return guarded([&]() -> int {
    if (check_handle(request)) return ISO_ERR_ARG;
    Request &r = *request;
    if (!r.send || !r.recv) return ISO_ERR_STATE;
    if (r.dirty) {
        if (r.started) {
            int rc = Iso_wait(request);
            if (rc != ISO_SUCCESS) return rc;
        }
        int rc = materialise(r);
        if (rc != ISO_SUCCESS) return rc;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const bool use_pdl = !r.knobs.no_pdl;
    if (r.wave_grid > 0) {
        // one cooperative launch that works through the (slab, launch) items
        WaveDev m{};
        m.launches = reinterpret_cast<const LaunchDev *>(static_cast<unsigned char *>(r.d_blob) + r.wave_launches_off);
        m.items = reinterpret_cast<const WaveItem *>(static_cast<unsigned char *>(r.d_blob) + r.wave_items_off);
        m.n = r.wave_items;
        m.done = r.d_counter;
        r.wave_run += 1;
        m.target = r.wave_run * (unsigned long long)r.wave_grid + (unsigned long long)r.skew_next;
        r.skew_next = 0;
        m.err = r.d_err;
        m.max_polls = r.wait_limit;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)r.wave_grid);
        cfg.blockDim = dim3(1024);
        cfg.dynamicSmemBytes = r.wave_smem;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        ISO_CUDA(cudaLaunchKernelEx(&cfg, iso_gather_rows_wave<kWideDepth>, m));
        r.last_stream = cuda_stream;
        r.started = true;
        return ISO_SUCCESS;
    }
    if (r.multi_grid > 0) {
        // all phases in one cooperative launch with grid barriers in between
        MultiDev m{};
        m.launches = reinterpret_cast<const LaunchDev *>(static_cast<unsigned char *>(r.d_blob) + r.multi_launches_off);
        m.n = (int)r.launches.size();
        m.counter = r.d_counter;
        m.epoch = r.epoch;
        m.err = r.d_err;
        m.max_polls = r.wait_limit;
        m.arrivals = (uint32_t)(r.multi_grid + r.skew_next);
        r.skew_next = 0;
        r.epoch += (unsigned long long)(m.n - 1) * (unsigned long long)r.multi_grid;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)r.multi_grid);
        cfg.blockDim = dim3(1024);
        cfg.dynamicSmemBytes = r.multi_smem;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        ISO_CUDA(cudaLaunchKernelEx(&cfg, iso_gather_rows_multi<kWideDepth>, m));
        r.last_stream = cuda_stream;
        r.started = true;
        return ISO_SUCCESS;
    }
    if (r.use_graph) {
        // replay of the captured launches (chains of slabs side by side when asked for)
        if (!r.graph_exec) {
            int rc = build_graph(r, use_pdl);
            if (rc != ISO_SUCCESS) return rc;
        }
        ISO_CUDA(cudaGraphLaunch(static_cast<cudaGraphExec_t>(r.graph_exec), stream));
        r.last_stream = cuda_stream;
        r.started = true;
        return ISO_SUCCESS;
    }
    if (r.slab_plan.size() > 1) {
        // slab after slab along dimension 0, all phases of a slab back to back: the slab's
        // intermediate blocks are read while they are still in L2, and every slab reuses the
        // same one-slab intermediate buffer, so those lines are overwritten in L2 instead of
        // being written back to device memory
        for (const auto &w : r.slab_plan)
            for (const LaunchPlan &L : r.launches) {
                int rc = launch_one(r, L, stream, use_pdl, w.first, w.second, w.first);
                if (rc != ISO_SUCCESS) return rc;
            }
        r.last_stream = cuda_stream;
        r.started = true;
        return ISO_SUCCESS;
    }
    for (const LaunchPlan &L : r.launches) {
        int rc = launch_one(r, L, stream, use_pdl);
        if (rc != ISO_SUCCESS) return rc;
    }
    r.last_stream = cuda_stream;
    r.started = true;
    return ISO_SUCCESS;
    });
}

int Iso_Start_host(Iso_request request, const void *host_sendbuf, void *host_recvbuf, void *cuda_stream)
{
    return guarded([&]() -> int {
    if (check_handle(request) || !host_sendbuf || !host_recvbuf) return ISO_ERR_ARG;
    Request &r = *request;
    if (!r.send || !r.recv) return ISO_ERR_STATE;
    const Comm &c = *r.comm;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (r.dirty) {
        if (r.started) {
            int rc = Iso_wait(request);
            if (rc != ISO_SUCCESS) return rc;
        }
        int rc = materialise(r);
        if (rc != ISO_SUCCESS) return rc;
    }
    const unsigned char *hs = static_cast<const unsigned char *>(host_sendbuf);
    unsigned char *hr = static_cast<unsigned char *>(host_recvbuf);
    std::vector<SlabPlan> slabs;
    if (r.multi_grid == 0 && r.wave_grid == 0) plan_slabs(r, slabs);
    // with a one-slab intermediate buffer the upload slabs must fit into it
    for (const SlabPlan &w : slabs)
        if (w.row_hi - w.row_lo > r.inter_rows) { slabs.clear(); break; }
    if (slabs.empty()) {
        // no pipelining possible: copy in, run, copy out
        const size_t sbytes = (size_t)(c.P * r.send_stride), rbytes = (size_t)(c.P * r.recv_stride);
        if (sbytes)
            ISO_CUDA(cudaMemcpyAsync(const_cast<unsigned char *>(r.send), hs, sbytes, cudaMemcpyHostToDevice, stream));
        int rc = Iso_Start(request, cuda_stream);
        if (rc != ISO_SUCCESS) return rc;
        if (rbytes) ISO_CUDA(cudaMemcpyAsync(hr, r.recv, rbytes, cudaMemcpyDeviceToHost, stream));
        r.host_timed = false;
        return ISO_SUCCESS;
    }

    // Pipelined over slabs of the leading dimension (enqueue_host_pipeline).  The same call
    // with the same host buffers is a fixed sequence of a few hundred copies, launches and
    // event operations: the first such call enqueues them one by one, the second captures
    // them into a graph, and from then on a start is one graph launch (submitting the
    // sequence one call at a time took longer than the 54 MB transfers of the 32^3 torus).
    const unsigned char *hs_b = hs;
    unsigned char *hr_b = hr;
    if (r.host_graph_exec && r.host_graph_hs == hs_b && r.host_graph_hr == hr_b) {
        ISO_CUDA(cudaGraphLaunch(static_cast<cudaGraphExec_t>(r.host_graph_exec), stream));
    } else if (r.knobs.host_graph && r.host_last_hs == hs_b && r.host_last_hr == hr_b && page_locked(hs_b) && page_locked(hr_b)) {
        if (r.host_graph_exec) cudaGraphExecDestroy(static_cast<cudaGraphExec_t>(r.host_graph_exec));
        r.host_graph_exec = nullptr;
        if (!r.host_main_stream)
            ISO_CUDA(cudaStreamCreateWithFlags(reinterpret_cast<cudaStream_t *>(&r.host_main_stream), cudaStreamNonBlocking));
        int rc = prepare_host_pipeline(r, slabs.size());
        if (rc != ISO_SUCCESS) return rc;
        cudaStream_t origin = static_cast<cudaStream_t>(r.host_main_stream);
        cudaGraph_t graph = nullptr;
        ISO_CUDA(cudaStreamBeginCapture(origin, cudaStreamCaptureModeThreadLocal));
        rc = enqueue_host_pipeline(r, slabs, hs_b, hr_b, origin, true);
        cudaError_t e = cudaStreamEndCapture(origin, &graph);
        cudaGraphExec_t exec = nullptr;
        if (rc == ISO_SUCCESS && e == cudaSuccess) e = cudaGraphInstantiate(&exec, graph, 0);
        if (graph) cudaGraphDestroy(graph);
        if (rc != ISO_SUCCESS) return rc;
        if (e != cudaSuccess) return cuda_fail(e);
        r.host_graph_exec = exec;
        r.host_graph_hs = hs_b;
        r.host_graph_hr = hr_b;
        ISO_CUDA(cudaGraphLaunch(exec, stream));
    } else {
        int rc = prepare_host_pipeline(r, slabs.size());
        if (rc == ISO_SUCCESS) rc = enqueue_host_pipeline(r, slabs, hs_b, hr_b, stream, false);
        if (rc != ISO_SUCCESS) return rc;
    }
    r.host_last_hs = hs_b;
    r.host_last_hr = hr_b;
    r.host_timed = true;
    r.host_slabs_used = (int)slabs.size();
    r.last_stream = cuda_stream;
    r.started = true;
    return ISO_SUCCESS;
    });
}

int Iso_wait(Iso_request request)
{
    return guarded([&]() -> int {
    if (check_handle(request)) return ISO_ERR_ARG;
    Request &r = *request;
    if (!r.started) return ISO_SUCCESS;
    cudaStream_t stream = static_cast<cudaStream_t>(r.last_stream);
    if (r.d_err && r.h_err) {
        ISO_CUDA(cudaMemcpyAsync(r.h_err, r.d_err, sizeof(int), cudaMemcpyDeviceToHost, stream));
    }
    ISO_CUDA(cudaStreamSynchronize(stream));
    if (r.h_err && *r.h_err) {
        *r.h_err = 0;
        ISO_CUDA(cudaMemsetAsync(r.d_err, 0, sizeof(int), stream));
        if (r.d_counter) {
            // a wait gave up: the arrival counters hold a partial count, start afresh
            ISO_CUDA(cudaMemsetAsync(r.d_counter, 0, (size_t)std::max(1, r.wave_counters) * sizeof(unsigned long long), stream));
            r.epoch = 0;
            r.wave_run = 0;
        }
        ISO_CUDA(cudaStreamSynchronize(stream));
        return ISO_ERR_TIMEOUT;
    }
    return ISO_SUCCESS;
    });
}

int Iso_request_get_host_transfer_ms(Iso_request request, float *upload_ms, float *download_ms, float *total_ms,
                                     int *slabs)
{
    return guarded([&]() -> int {
    if (check_handle(request)) return ISO_ERR_ARG;
    Request &r = *request;
    if (!r.host_timed) return ISO_ERR_STATE;
    int rc = Iso_wait(request);
    if (rc != ISO_SUCCESS) return rc;
    auto span = [&](int a, int b, float *out) -> cudaError_t {
        if (!out) return cudaSuccess;
        return cudaEventElapsedTime(out, static_cast<cudaEvent_t>(r.host_timing[a]), static_cast<cudaEvent_t>(r.host_timing[b]));
    };
    ISO_CUDA(span(0, 1, upload_ms));
    ISO_CUDA(span(2, 3, download_ms));
    ISO_CUDA(span(4, 5, total_ms));
    if (slabs) *slabs = r.host_slabs_used;
    return ISO_SUCCESS;
    });
}

int Iso_request_check_guards(Iso_request request, int64_t *violations)
{
    return guarded([&]() -> int {
    if (check_handle(request) || !violations) return ISO_ERR_ARG;
    Request &r = *request;
    if (r.started) {
        int rc = Iso_wait(request);
        if (rc != ISO_SUCCESS && rc != ISO_ERR_TIMEOUT) return rc;
    }
    int64_t bad = 0;
    if (r.d_inter_alloc) {
        std::vector<unsigned char> band(2 * kGuardBytes);
        ISO_CUDA(cudaMemcpy(band.data(), r.d_inter_alloc, kGuardBytes, cudaMemcpyDeviceToHost));
        ISO_CUDA(cudaMemcpy(band.data() + kGuardBytes, r.d_inter + r.d_inter_bytes, kGuardBytes, cudaMemcpyDeviceToHost));
        for (unsigned char b : band) bad += b != (unsigned char)kGuardPattern;
    }
    *violations = bad;
    return ISO_SUCCESS;
    });
}

int Iso_request_set_wait_limit(Iso_request request, unsigned int polls)
{
    if (check_handle(request) || polls == 0) return ISO_ERR_ARG;
    request->wait_limit = polls;
    return ISO_SUCCESS;
}

int Iso_request_test_skew_arrivals(Iso_request request, int extra)
{
    if (check_handle(request) || extra < 0 || extra > 1024) return ISO_ERR_ARG;
    request->skew_next = extra;
    return ISO_SUCCESS;
}

int Iso_measure_launch_floor(void *cuda_stream, int launches, int dependent, float *microseconds_per_launch)
{
    return guarded([&]() -> int {
    if (launches < 1 || launches > (1 << 20) || !microseconds_per_launch) return ISO_ERR_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaEvent_t t0 = nullptr, t1 = nullptr;
    ISO_CUDA(cudaEventCreate(&t0));
    cudaError_t e = cudaEventCreate(&t1);
    auto one = [&]() -> cudaError_t {
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(1);
        cfg.blockDim = dim3(32);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = dependent ? 1 : 0;
        return cudaLaunchKernelEx(&cfg, iso_empty_kernel, 0);
    };
    for (int k = 0; k < 16 && e == cudaSuccess; ++k) e = one();
    if (e == cudaSuccess) e = cudaEventRecord(t0, stream);
    for (int k = 0; k < launches && e == cudaSuccess; ++k) e = one();
    if (e == cudaSuccess) e = cudaEventRecord(t1, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    float ms = 0.0f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, t0, t1);
    cudaEventDestroy(t0);
    if (t1) cudaEventDestroy(t1);
    if (e != cudaSuccess) return cuda_fail(e);
    *microseconds_per_launch = ms * 1e3f / (float)launches;
    return ISO_SUCCESS;
    });
}

int Iso_request_get_stats(Iso_request request, Iso_stats *out)
{
    if (check_handle(request) || !out) return ISO_ERR_ARG;
    *out = request->stats;
    if (!request->dirty && (request->multi_grid > 0 || request->wave_grid > 0)) out->launches = 1;
    else if (!request->dirty && request->slab_plan.size() > 1) out->launches *= (int)request->slab_plan.size();
    return ISO_SUCCESS;
}

int Iso_request_get_parts(Iso_request request, Iso_part *out, int capacity, int *count)
{
    return guarded([&]() -> int {
    if (check_handle(request) || !count || capacity < 0 || (capacity > 0 && !out)) return ISO_ERR_ARG;
    int n = 0;
    std::vector<const LaunchPlan *> plans;
    for (const LaunchPlan &L : request->launches) {
        plans.push_back(&L);
        for (const LaunchPlan &S : L.side) plans.push_back(&S);
    }
    for (const LaunchPlan *plan : plans) {
        const LaunchPlan &L = *plan;
        for (const LoweredPart &lp : L.parts) {
            if (n < capacity) {
                Iso_part q{};
                q.phase = lp.p.phase;
                q.round = lp.p.round;
                q.slot = lp.p.slot;
                q.src_buf = lp.p.src_buf;
                q.dst_buf = lp.p.dst_buf;
                q.kernel = L.kernel;
                q.width = lp.width;
                q.src_off = lp.p.src_off;
                q.dst_off = lp.p.dst_off;
                q.len = lp.p.len;
                std::memcpy(q.shift, lp.p.shift, sizeof(q.shift));
                std::memcpy(q.check, lp.p.check, sizeof(q.check));
                out[n] = q;
            }
            ++n;
        }
    }
    *count = n;
    return ISO_SUCCESS;
    });
}

int Iso_request_free(Iso_request *request)
{
    if (!request || !*request) return ISO_ERR_ARG;
    Iso_request_s *r = *request;
    int rc = ISO_SUCCESS;
    if (r->started) rc = Iso_wait(r);
    release_device(*r);
    comm_unref(r->comm);
    delete r;
    *request = nullptr;
    return rc == ISO_ERR_TIMEOUT ? ISO_SUCCESS : rc;
}

const char *Iso_error_string(int code)
{
    switch (code) {
    case ISO_SUCCESS: return "success";
    case ISO_ERR_ARG: return "invalid argument";
    case ISO_ERR_DIMS: return "invalid torus dimensions";
    case ISO_ERR_COUNT: return "block sizes do not match or overflow";
    case ISO_ERR_ALIGN: return "unsupported alignment";
    case ISO_ERR_NOMEM: return "out of memory";
    case ISO_ERR_CUDA: return "CUDA call failed";
    case ISO_ERR_OVERLAP: return "buffers or blocks overlap";
    case ISO_ERR_STATE: return "call not valid in this state";
    case ISO_ERR_TIMEOUT: return "a bounded wait inside a kernel expired";
    case ISO_ERR_TOO_LARGE: return "problem does not fit the static scratch area";
    default: return "unknown error code";
    }
}

int Iso_last_cuda_error(void) { return g_last_cuda_error; }

int Iso_selftest(void)
{
    // exact division by multiplication: edge values and a pseudo-random sweep
    const uint32_t divisors[] = {1, 2, 3, 5, 7, 9, 10, 36, 81, 162, 255, 256, 257, 1000, 1280, 6144, 65535, 65536, 65537,
                                 1000003, 0x7fffffffu, 0x80000000u, 0xfffffffeu, 0xffffffffu};
    uint64_t x = 88172645463325252ull;
    for (uint32_t d : divisors) {
        FastDiv f = make_fastdiv(d);
        const uint32_t edges[] = {0, 1, d - 1, d, d + 1, 2 * d - 1, 2 * d, 0x7fffffffu, 0x80000000u, 0xffffffffu};
        for (uint32_t n : edges)
            if (fastdiv_host(f, n) != n / d) return ISO_ERR_STATE;
        for (int k = 0; k < 20000; ++k) {
            x ^= x << 13; x ^= x >> 7; x ^= x << 17;
            uint32_t n = (uint32_t)(x >> 16);
            if (fastdiv_host(f, n) != n / d) return ISO_ERR_STATE;
        }
    }
    return ISO_SUCCESS;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------
// Allocation-free variant of the message-combining all-to-all.
//
// Some programs may not allocate device memory at the point where they need the collective:
// a solver whose memory budget was fixed and handed out at start-up, a plug-in that runs
// inside another framework's memory pool, or a service that forbids cudaMalloc on its hot
// path because the call synchronises the whole device.  The ordinary path (Iso_neighbor_alltoall_init +
// Iso_Start) allocates its index tables and its intermediate buffer with cudaMalloc.  The
// entry point below keeps both in a fixed array that is part of the library image
// instead, so that it never allocates; the price is an upper bound on the problem size and
// one shared scratch area per device.
namespace {

// The scratch area: intermediate buffer first, unit tables behind it.  Every device that
// loads the library holds one copy until the process exits.
static __device__ __align__(256) unsigned char iso_static_scratch[ISO_STATIC_SCRATCH_BYTES];

// Device address of the scratch area per device ordinal.  The array's name is only a
// host-side handle; kernels need the address cudaGetSymbolAddress returns on that device.
constexpr int kMaxDevices = 64;
unsigned char *g_scratch_addr[kMaxDevices] = {nullptr};

int scratch_for_current_device(unsigned char **out)
{
    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return cuda_fail(e);
    if (device < 0 || device >= kMaxDevices) return ISO_ERR_ARG;
    static std::mutex guard;  // two host threads may make their first call at the same time
    std::lock_guard<std::mutex> lock(guard);
    if (!g_scratch_addr[device]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, iso_static_scratch);
        if (e != cudaSuccess) return cuda_fail(e);
        if (!p) return ISO_ERR_CUDA;
        g_scratch_addr[device] = static_cast<unsigned char *>(p);
    }
    *out = g_scratch_addr[device];
    return ISO_SUCCESS;
}

int64_t round_up_256(int64_t x) { return (x + 255) / 256 * 256; }

}  // namespace

extern "C" int Iso_neighbor_alltoall_static(int d, const int dims[], int s, const int relative_coordinates[],
                                            const void *sendbuf, void *recvbuf, int count, Iso_datatype type,
                                            void *cuda_stream)
{
    return guarded([&]() -> int {
    if (!dims || s < 0 || (s > 0 && !relative_coordinates) || !sendbuf || !recvbuf || count < 0 || type < 1)
        return ISO_ERR_ARG;
    if (d < 1 || d > ISO_MAX_DIMS) return ISO_ERR_DIMS;

    // the neighbourhood and the request live on the host stack / heap for this call only
    Comm comm;
    comm.d = d;
    comm.s = s;
    int64_t P = 1, stride = 1;
    for (int j = 0; j < d; ++j) {
        if (dims[j] < 1 || P > (int64_t)0x7fffffff / dims[j]) return ISO_ERR_DIMS;
        P *= dims[j];
    }
    comm.P = P;
    for (int j = d - 1; j >= 0; --j) {
        comm.dims[j] = dims[j];
        comm.periodic[j] = 1;
        comm.rank_stride[j] = stride;
        stride *= dims[j];
    }
    comm.coords.assign(relative_coordinates, relative_coordinates + (size_t)s * d);

    const int64_t m = (int64_t)count * type;
    Request r;
    r.comm = &comm;
    r.knobs = read_knobs();
    r.kind = ISO_KIND_ALLTOALL;
    r.alg = ISO_ALG_COMBINING;
    r.fusion = 1;
    r.layout = ISO_LAYOUT_PACKED;
    r.bulk_threshold_asked = 0;  // vector kernel only: no error flag, nothing that must start at zero
    r.send = static_cast<const unsigned char *>(sendbuf);
    r.recv = static_cast<unsigned char *>(recvbuf);
    r.s = s;
    r.len.assign(s, m);
    r.sdispl.resize(s);
    r.rdispl.resize(s);
    for (int i = 0; i < s; ++i) r.sdispl[i] = r.rdispl[i] = (int64_t)i * m;
    r.send_stride = r.recv_stride = (int64_t)s * m;
    if (s == 0 || m == 0) return ISO_SUCCESS;
    if (r.send_stride > INT64_MAX / P) return ISO_ERR_COUNT;
    {
        const unsigned char *s0 = r.send, *s1 = r.send + P * r.send_stride;
        const unsigned char *d0 = r.recv, *d1 = r.recv + P * r.recv_stride;
        if (s0 < d1 && d0 < s1) return ISO_ERR_OVERLAP;
    }
    int rc = build_schedule(r);
    if (rc != ISO_SUCCESS) return rc;

    // does it fit?  (checked before anything touches the device)
    if (r.inter_stride > (int64_t)ISO_STATIC_SCRATCH_BYTES / P) return ISO_ERR_TOO_LARGE;
    const int64_t inter_bytes = round_up_256(P * r.inter_stride);
    unsigned char *scratch = nullptr;
    rc = scratch_for_current_device(&scratch);
    if (rc != ISO_SUCCESS) return rc;
    int device = 0, sms = 0;
    if (cudaGetDevice(&device) == cudaSuccess &&
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) == cudaSuccess && sms > 0)
        r.sm_count = sms;
    rc = lower_schedule(r, (uintptr_t)r.send, (uintptr_t)r.recv, (uintptr_t)scratch);
    if (rc != ISO_SUCCESS) return rc;
    int64_t table_bytes = 0;
    for (LaunchPlan &L : r.launches) {
        if (L.kernel != KERNEL_VEC) return ISO_ERR_STATE;
        L.units_off = (size_t)table_bytes;
        table_bytes += (int64_t)L.units_per_proc * (int64_t)sizeof(UnitDev);
    }
    if (inter_bytes + table_bytes > (int64_t)ISO_STATIC_SCRATCH_BYTES) return ISO_ERR_TOO_LARGE;

    // unit tables, built on the host and copied behind the intermediate buffer
    std::vector<unsigned char> blob((size_t)table_bytes, 0);
    for (const LaunchPlan &L : r.launches) fill_units(r, L, reinterpret_cast<UnitDev *>(blob.data() + L.units_off));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    unsigned char *tables = scratch + inter_bytes;
    // The copy reads `blob`, which dies with this call: outside a stream capture the runtime
    // has staged a pageable source by the time the call returns, inside one the graph would
    // keep the dangling host pointer - hence no call of this function inside a capture.
    if (table_bytes > 0)
        ISO_CUDA(cudaMemcpyAsync(tables, blob.data(), (size_t)table_bytes, cudaMemcpyHostToDevice, stream));

    // the ordinary launch path, pointed at the scratch area (nothing here is owned by `r`)
    r.d_blob = tables;
    r.d_inter = scratch;
    for (const LaunchPlan &L : r.launches) {
        rc = launch_one(r, L, stream, false);
        if (rc != ISO_SUCCESS) return rc;
    }
    return ISO_SUCCESS;
    });
}
