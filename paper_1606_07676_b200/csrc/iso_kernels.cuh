// Device code of the isomorphic neighbourhood collectives (sm_100a).
//
// One launch applies a list of parts to every process (paper, Section V: in a round all
// processes forward the same relative blocks): for process r and part t
//     dst_buf[r] + dst_off_t .. + len_t  =  src_buf[r (-) shift_t] + src_off_t .. + len_t
// Packing, "sending" and unpacking of a combined message are this single gather; nothing
// is staged through memory in between (the zero-copy goal of Section III-C).
//
// Work decomposition shared by both kernels: a CTA owns a tile of consecutive processes.
// The payload of one process in this launch is cut into units (vector kernel: `width`
// bytes; bulk kernel: chunks of up to `width` bytes); unit u of tile-local process q has
// the flat index q * units_per_proc + u, and consecutive threads take consecutive flat
// indices, so a warp touches consecutive bytes of one part (or of neighbouring parts)
// whatever the block size is.
#pragma once

#include <cstdint>

#include "iso.h"

namespace iso {

struct FastDivDev {
    uint32_t m, s1, s2, div;
};

struct alignas(16) PartDev {
    long long src_off;     // byte offset inside a process's source buffer
    long long dst_off;     // byte offset inside the own destination buffer
    long long len;         // bytes
    long long rank_delta;  // source rank = own rank + rank_delta (+ wrap corrections)
    uint32_t first_unit;   // index of the part's first unit among the launch's units
    uint32_t units;
    uint8_t src_buf, dst_buf, nnz, pad0;
    uint8_t dim[ISO_MAX_DIMS];  // index into the launch's used dimensions
    int32_t c[ISO_MAX_DIMS];    // coordinate shift along that dimension
    uint32_t pad1;
};

// Everything the vector kernel needs to know about one unit position of a process's payload.
struct alignas(16) UnitDev {
    long long src_term;  // rank_delta * source stride + source offset of the unit (bytes)
    long long dst_term;  // destination offset of the unit (bytes)
    // Dense form (nnz = the launch's n_used, dim[e] = e): c[e] is the coordinate shift
    // along used dimension e, 0 for none.  Compact form: only the shifted dimensions are
    // listed, c[e] != 0 along used dimension dim[e] for e < nnz.
    int32_t c[ISO_MAX_DIMS];
    uint8_t src_buf, dst_buf, nnz;
    uint8_t width;  // bytes of this unit: 1, 2, 4, 8 or 16 (launches of mixed unit widths; otherwise the launch's width)
    uint8_t dim[ISO_MAX_DIMS];
    uint8_t pad1[4];
};
static_assert(sizeof(UnitDev) == 64, "unit descriptors are read as four 16-byte words");

struct LaunchDev {
    const PartDev *parts;
    const UnitDev *units;    // vector kernel: one entry per unit position
    const uint16_t *lookup;  // unit >> lookup_shift -> part (unused when uniform_units > 0)
    unsigned char *buf[3];   // send, recv, inter
    long long buf_stride[3];
    long long P;
    long long row_lo, row_hi;  // the processes this launch works on: ranks [row_lo, row_hi)
    int *err;                // device error flag (bulk kernel time-outs)
    uint32_t nparts;
    uint32_t units_per_proc;
    uint32_t uniform_units;
    uint32_t lookup_shift;
    uint32_t width;          // bytes per unit / chunk
    uint32_t chunk_units;    // vector kernel: unit positions owned by one row slot of a CTA
    uint32_t rows_per_pass;  // vector kernel: rows a CTA works on at the same time
    int tile_procs;
    int n_used;
    int mesh_mask;           // bit k set: used dimension k is not periodic
    int grid_share;          // host side only: launches of this kind that run side by side
    uint32_t tab_iters;      // coordinate table: row groups a CTA visits at most (0: no table)
    uint32_t tab_stride;     // coordinate table: 32-bit words per row (4 or 8)
    uint32_t side_offset;    // hybrid kernel, bulk side: byte offset of its staging area in shared memory
    uint32_t col_split;      // vector kernel: column chunks the CTAs are dealt to (0 or 1: a CTA covers whole rows)
    uint32_t keep_inter;     // vector kernel, 16-byte units: stores into the intermediate buffer ask the L2 to evict them last
    FastDivDev div_units;    // division by units_per_proc
    FastDivDev div_uniform;  // division by uniform_units
    int used_dim[ISO_MAX_DIMS];
    uint32_t used_size[ISO_MAX_DIMS];       // p_j of the used dimensions
    long long used_rstride[ISO_MAX_DIMS];   // ranks per step along the used dimensions
    uint32_t used_wrap[ISO_MAX_DIMS];       // p_j * rank stride: added when a shift wraps around
    FastDivDev div_rstride[ISO_MAX_DIMS];   // division by the rank stride of a used dimension
    FastDivDev div_size[ISO_MAX_DIMS];      // division by the size of a used dimension
};

__device__ __forceinline__ uint32_t fastdiv(const FastDivDev &f, uint32_t n)
{
    uint32_t t = __umulhi(f.m, n);
    return (t + ((n - t) >> f.s1)) >> f.s2;
}

// Coordinates (along the dimensions this launch shifts in) of the tile's processes.
__device__ __forceinline__ void tile_coordinates(const LaunchDev &L, long long r0, int np, uint32_t *s_coord)
{
    // ranks are below 2^31, so the exact 32-bit division applies
    for (int k = 0; k < L.n_used; ++k)
        for (int q = threadIdx.x; q < np; q += blockDim.x) {
            const uint32_t x = fastdiv(L.div_rstride[k], (uint32_t)(r0 + q));
            s_coord[k * L.tile_procs + q] = x - fastdiv(L.div_size[k], x) * L.used_size[k];
        }
}

struct UnitAddr {
    const unsigned char *src;
    unsigned char *dst;
    uint32_t bytes;  // bytes of this unit (bulk kernel: the last chunk of a part is shorter)
    bool valid;      // false: the source lies outside a non-periodic dimension
};

// Decodes flat unit index `id` of the tile into addresses.
__device__ __forceinline__ UnitAddr decode_unit(const LaunchDev &L, long long r0, uint32_t id,
                                                const uint32_t *s_coord)
{
    const uint32_t q = fastdiv(L.div_units, id);
    const uint32_t u = id - q * L.units_per_proc;
    uint32_t t;
    if (L.uniform_units) {
        t = fastdiv(L.div_uniform, u);
    } else {
        t = L.lookup[u >> L.lookup_shift];
        while (t + 1 < L.nparts && __ldg(&L.parts[t + 1].first_unit) <= u) ++t;
    }
    const PartDev *p = L.parts + t;
    const uint32_t k = u - __ldg(&p->first_unit);
    long long rs = r0 + q + __ldg(&p->rank_delta);
    bool valid = true;
    const int nnz = __ldg(&p->nnz);
    for (int e = 0; e < nnz; ++e) {
        const int dk = __ldg(&p->dim[e]);
        const int c = __ldg(&p->c[e]);
        const int x = (int)s_coord[dk * L.tile_procs + q];
        if (L.mesh_mask >> dk & 1) {
            const int y = x - c;
            valid = valid && y >= 0 && y < (int)L.used_size[dk];
        } else if (x < c) {
            rs += (long long)L.used_size[dk] * L.used_rstride[dk];
        }
    }
    const long long within = (long long)k * L.width;
    const long long len = __ldg(&p->len);
    UnitAddr a;
    a.src = L.buf[__ldg(&p->src_buf)] + rs * L.buf_stride[__ldg(&p->src_buf)] + __ldg(&p->src_off) + within;
    a.dst = L.buf[__ldg(&p->dst_buf)] + (r0 + q) * L.buf_stride[__ldg(&p->dst_buf)] + __ldg(&p->dst_off) + within;
    const long long rest = len - within;
    a.bytes = (uint32_t)(rest < (long long)L.width ? rest : (long long)L.width);
    a.valid = valid;
    return a;
}

template <int W> struct VecOf;
template <> struct VecOf<0> { using type = uint4; };  // mixed widths: slots of the widest unit
template <> struct VecOf<16> { using type = uint4; };
template <> struct VecOf<8> { using type = uint2; };
template <> struct VecOf<4> { using type = uint32_t; };
template <> struct VecOf<2> { using type = uint16_t; };
template <> struct VecOf<1> { using type = uint8_t; };

// Programmatic dependent launch: `grid_dependency_wait` blocks until the preceding kernel
// in the stream has completed and its writes are visible; everything before it (tables,
// coordinates) overlaps with that kernel's tail.  Both are no-ops for ordinary launches.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <int W> __device__ __forceinline__ void cp_async(void *smem_dst, const void *gsrc);
template <> __device__ __forceinline__ void cp_async<16>(void *smem_dst, const void *gsrc)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
                 : "memory");
}
template <> __device__ __forceinline__ void cp_async<8>(void *smem_dst, const void *gsrc)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
                 : "memory");
}
template <> __device__ __forceinline__ void cp_async<4>(void *smem_dst, const void *gsrc)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
                 : "memory");
}
// W = 0: the width is the unit's own (1, 2, 4, 8 or 16 bytes), known only at run time.
// `w` holds the width in its low byte and, for 1- and 2-byte units, the unit's offset inside
// its aligned 4-byte word in the next one: cp.async moves at least 4 bytes, so such a unit
// fetches the whole word (rows start on 4-byte boundaries in these launches, so the word
// lies inside the same row) and stores only its own bytes.
template <int W> __device__ __forceinline__ void cp_async_unit(void *smem_dst, const unsigned char *gsrc, uint32_t w)
{
    if (W != 0) {
        cp_async<(W != 0 ? W : 16)>(smem_dst, gsrc);
    } else if ((w & 0xff) == 16) {
        cp_async<16>(smem_dst, gsrc);
    } else if ((w & 0xff) == 8) {
        cp_async<8>(smem_dst, gsrc);
    } else if ((w & 0xff) == 4) {
        cp_async<4>(smem_dst, gsrc);
    } else {
        cp_async<4>(smem_dst, gsrc - (w >> 8));
    }
}
template <int W> __device__ __forceinline__ void store_unit(unsigned char *dst, const typename VecOf<W>::type *slot, uint32_t w)
{
    if (W != 0) {
        *reinterpret_cast<typename VecOf<W>::type *>(dst) = *slot;
    } else if ((w & 0xff) == 16) {
        *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(slot);
    } else if ((w & 0xff) == 8) {
        *reinterpret_cast<uint2 *>(dst) = *reinterpret_cast<const uint2 *>(slot);
    } else if ((w & 0xff) == 4) {
        *reinterpret_cast<uint32_t *>(dst) = *reinterpret_cast<const uint32_t *>(slot);
    } else {
        const uint32_t word = *reinterpret_cast<const uint32_t *>(slot) >> (8 * (w >> 8));
        if ((w & 0xff) == 2) *reinterpret_cast<uint16_t *>(dst) = (uint16_t)word;
        else *dst = (uint8_t)word;
    }
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// L2 eviction priority for the blocks a slab keeps for its next phase: written with the
// evict_last policy they outlast the streamed send and receive lines around them, are read
// back out of the L2 and are overwritten there by the next slab instead of being written
// back to device memory in between.  A hint only: the data path is the same store.
__device__ __forceinline__ uint64_t l2_policy_evict_last()
{
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}
__device__ __forceinline__ void store_16_hinted(unsigned char *dst, const uint4 &v, uint64_t policy)
{
    asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w),
                 "l"(policy)
                 : "memory");
}

// What a thread keeps about the unit position it owns.
struct UnitRegs {
    const unsigned char *A;  // source base: buffer + src_term
    unsigned char *B;        // destination base: buffer + dst_term
    long long stride_s, stride_d;
    int c[ISO_MAX_DIMS];
    uint32_t nnz;
    uint32_t width;
    uint32_t dims_lo, dims_hi;  // dim[0..3], dim[4..7], one byte each
    bool to_inter;              // the destination is the intermediate buffer
};

__device__ __forceinline__ UnitRegs load_unit(const LaunchDev &L, uint32_t u)
{
    const uint4 *raw = reinterpret_cast<const uint4 *>(L.units + u);
    const uint4 a = __ldg(raw), b = __ldg(raw + 1), c = __ldg(raw + 2), d = __ldg(raw + 3);
    UnitRegs R;
    const long long src_term = (long long)(((unsigned long long)a.y << 32) | a.x);
    const long long dst_term = (long long)(((unsigned long long)a.w << 32) | a.z);
    const int sb = d.x & 0xff, db = (d.x >> 8) & 0xff;
    R.A = L.buf[sb] + src_term;
    R.B = L.buf[db] + dst_term;
    R.stride_s = L.buf_stride[sb];
    R.stride_d = L.buf_stride[db];
    R.c[0] = (int)b.x; R.c[1] = (int)b.y; R.c[2] = (int)b.z; R.c[3] = (int)b.w;
    R.c[4] = (int)c.x; R.c[5] = (int)c.y; R.c[6] = (int)c.z; R.c[7] = (int)c.w;
    R.nnz = (d.x >> 16) & 0xff;
    R.to_inter = db == 2;  // ISO_BUF_INTER
    R.width = d.x >> 24;
    if (R.width < 4) R.width |= ((uint32_t)(uintptr_t)R.A & 3u) << 8;  // offset inside the aligned word
    R.dims_lo = d.y;
    R.dims_hi = d.z;
    return R;
}

// Vector gather.  Thread t of a CTA owns one unit position (row slot g = t / chunk_units,
// unit u = t % chunk_units): it loads that unit's descriptor once and then walks down its
// rows (processes) with running source and destination pointers.  CTA b takes the row
// groups b, b + grid, b + 2*grid, ... (a row group is rows_per_pass consecutive rows), so
// that at any moment the CTAs of the grid work on one contiguous window of processes, as a
// plain copy kernel would, instead of on `grid` separate streams (measured: 42 against 48
// microseconds per all-to-all on the 32^3 torus).  Per row the work is a wrap test per
// shifted dimension - the row's coordinate by exact 32-bit division - and two pointer
// increments.
//
// W = 0 is a launch of mixed unit widths (every unit 1, 2, 4, 8 or 16 bytes wide, as its
// descriptor says): the ragged rows of the irregular collectives then take one launch per
// phase instead of one per width, and pieces that share a 32-byte sector are moved at the
// same time by the same CTA.
//
// Data path for W in {16, 8, 4}: cp.async from global memory into a thread-private ring of
// DEPTH slots in shared memory, so that DEPTH loads per thread are in flight without
// holding registers; a slot is read back and stored to its destination as soon as the
// oldest group has landed, and refilled with the load of DEPTH rows ahead.
//
// NU is the number of shifted dimensions per unit the kernel is compiled for (dense
// descriptors: the launch's n_used must not exceed it; compact descriptors: no unit's nnz
// may; ISO_MAX_DIMS is the general case), MESH whether some dimensions are non-periodic
// (then a row whose source lies outside the mesh is skipped).  COMPACT selects the compact
// descriptor form: a launch that shifts along many dimensions, each unit along few of
// them (the last phase of a schedule whose final hops were postponed, the direct schedule
// in high dimension), then tests per row only the dimensions its unit moves along.
//
// TAB: the coordinates of the rows come from a table in shared memory instead of two exact
// divisions per row, dimension and THREAD.  All threads of a row slot walk the same rows, so
// the CTA computes the coordinates of every row it will visit once, before it orders itself
// behind the previous kernel (the table depends on nothing that kernel writes), and a thread
// then reads its row's entry with one shared-memory load.  The direct schedule, three wrap
// tests per row, spent 110 instructions per 16-byte unit and ran at 70 % issue utilisation
// with the integer-multiply pipe as the top stall; the table removes that arithmetic.
template <int W, int DEPTH, int NU, bool MESH, bool COMPACT, bool TAB = false>
__device__ __forceinline__ void gather_rows_body(const LaunchDev &L, unsigned char *ring_base, bool dependent_launch,
                                                 uint32_t cta, uint32_t n_cta, const uint32_t nthr)
{   // nthr: threads of the CTA that run this body (all of them, except in the hybrid kernel)
    using V = typename VecOf<W>::type;
    V *const ring = reinterpret_cast<V *>(ring_base) + threadIdx.x;  // slot k at ring[k * nthr]
    V *const ring_end = ring + DEPTH * nthr;

    const uint32_t CU = L.chunk_units, U = L.units_per_proc;
    const int G = (int)L.rows_per_pass;
    const int g = (int)(threadIdx.x / CU);
    // Rows longer than a CTA (col_split = n > 1): instead of covering a row in n passes - each
    // a fresh ramp and drain of the ring over the few rows a CTA has - the CTAs are dealt to n
    // column chunks: CTA b owns chunk b mod n and takes every (grid / n)-th row, in one pass.
    const uint32_t ncol = L.col_split > 1 ? L.col_split : 1;
    const uint32_t col = cta % ncol;
    cta /= ncol;
    n_cta /= ncol;
    const uint32_t ul = threadIdx.x - (uint32_t)g * CU + col * CU;
    const long long r0 = L.row_lo + (long long)G * cta + g;
    const bool active = g < G && r0 < L.row_hi && ul < U && threadIdx.x < (uint32_t)G * CU;
    const long long rstep = (long long)G * n_cta;
    // the tables are not produced by kernels: fetch the first descriptor before ordering
    // behind the previous kernel
    UnitRegs R_first;
    if (active) R_first = load_unit(L, ul);
    // entry (it * G + g) of the coordinate table: row slot g in the CTA's it-th row group
    uint32_t *const tab = reinterpret_cast<uint32_t *>(ring_base + (size_t)DEPTH * nthr * sizeof(V));
    const uint32_t NT = TAB ? L.tab_stride : 0;
    if (TAB) {
        const long long group0 = L.row_lo + (long long)G * cta;
        const uint32_t entries = L.tab_iters * (uint32_t)G;
        for (uint32_t j = threadIdx.x; j < entries; j += nthr) {
            const uint32_t it = j / (uint32_t)G;
            const long long r = group0 + (long long)it * rstep + (j - it * (uint32_t)G);
            if (r < L.row_hi) {
                for (int k = 0; k < L.n_used; ++k) {
                    const uint32_t t = fastdiv(L.div_rstride[k], (uint32_t)r);
                    tab[j * NT + k] = t - fastdiv(L.div_size[k], t) * L.used_size[k];
                }
            }
        }
        __syncthreads();
    }
    if (dependent_launch) {
        grid_dependency_wait();
        grid_launch_dependents();
    }
    if (!active) return;
    const long long r_end = L.row_hi;
    const uint32_t tab_step = (uint32_t)G * NT;

    for (uint32_t u = ul; u < U; u += (ncol > 1 ? U : CU)) {
        const UnitRegs R = u == ul ? R_first : load_unit(L, u);
        // used dimension tested in position e: e itself (dense) or the unit's own list
        auto dim_of = [&](int e) -> int {
            return COMPACT ? (int)(((e < 4 ? R.dims_lo : R.dims_hi) >> (8 * (e & 3))) & 0xffu) : e;
        };
        const int n_tests = COMPACT ? (int)R.nnz : L.n_used;
        long long wrap_bytes[NU > 0 ? NU : 1];
#pragma unroll
        for (int e = 0; e < NU; ++e) wrap_bytes[e] = (long long)L.used_wrap[dim_of(e)] * R.stride_s;
        const long long src_step = rstep * R.stride_s, dst_step = rstep * R.stride_d;
        const bool keep = W == 16 && L.keep_inter && R.to_inter;
        const uint64_t policy = keep ? l2_policy_evict_last() : 0;

        // `row`: the row's entry of the coordinate table (TAB), unused otherwise
        auto source = [&](const unsigned char *nowrap, long long r, const uint32_t *row, const unsigned char *&src) -> bool {
            bool valid = true;
            src = nowrap;
            uint4 xs = make_uint4(0, 0, 0, 0);
            if (TAB && !COMPACT && NU >= 1 && NU <= 4) xs = *reinterpret_cast<const uint4 *>(row);
#pragma unroll
            for (int e = 0; e < NU; ++e) {
                if ((!COMPACT && NU < ISO_MAX_DIMS) || e < n_tests) {
                    const int k = dim_of(e);
                    int x;
                    if (TAB && !COMPACT && NU <= 4) {
                        x = (int)(e == 0 ? xs.x : (e == 1 ? xs.y : (e == 2 ? xs.z : xs.w)));
                    } else if (TAB) {
                        x = (int)row[k];
                    } else {
                        const uint32_t t = fastdiv(L.div_rstride[k], (uint32_t)r);
                        x = (int)(t - fastdiv(L.div_size[k], t) * L.used_size[k]);
                    }
                    if (MESH && ((L.mesh_mask >> k) & 1)) {
                        const int y = x - R.c[e];
                        valid = valid && y >= 0 && y < (int)L.used_size[k];
                    } else if (x < R.c[e]) {
                        src += wrap_bytes[e];
                    }
                }
            }
            return valid;
        };

        long long r_ld = r0;
        const unsigned char *src_ld = R.A + r0 * R.stride_s;
        unsigned char *dst = R.B + r0 * R.stride_d;
        const uint32_t *row_ld = tab + (uint32_t)g * NT, *row_st = row_ld;
#pragma unroll
        for (int i = 0; i < DEPTH; ++i) {
            if (r_ld < r_end) {
                const unsigned char *src;
                if (source(src_ld, r_ld, row_ld, src)) cp_async_unit<W>(ring + i * nthr, src, R.width);
                r_ld += rstep;
                src_ld += src_step;
                row_ld += tab_step;
            }
            cp_async_commit();
        }
        V *slot = ring;
        for (long long r = r0; r < r_end; r += rstep) {
            cp_async_wait<DEPTH - 1>();
            bool valid = true;
            if (MESH) {
                const unsigned char *ignored;
                valid = source(nullptr, r, row_st, ignored);
                row_st += tab_step;
            }
            if (W == 16 && keep) {
                if (valid) store_16_hinted(dst, *reinterpret_cast<const uint4 *>(slot), policy);
            } else if (valid) {
                store_unit<W>(dst, slot, R.width);
            }
            dst += dst_step;
            if (r_ld < r_end) {
                const unsigned char *src;
                if (source(src_ld, r_ld, row_ld, src)) cp_async_unit<W>(slot, src, R.width);
                r_ld += rstep;
                src_ld += src_step;
                row_ld += tab_step;
            }
            cp_async_commit();
            slot += nthr;
            if (slot == ring_end) slot = ring;
        }
        cp_async_wait<0>();
    }
}

template <int W, int DEPTH, int NU, bool MESH, bool COMPACT>
__global__ void __launch_bounds__(256, 4) iso_gather_rows(const __grid_constant__ LaunchDev L)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    gather_rows_body<W, DEPTH, NU, MESH, COMPACT>(L, smem_raw, true, blockIdx.x, gridDim.x, blockDim.x);
}

// The same body in CTAs of up to 1024 threads, for launches whose payload per process has
// more than 256 unit positions: one CTA then covers up to 16 KB of a row at a time, so rows
// are still visited one after the other instead of in 4 KB columns.
template <int W, int DEPTH, int NU, bool MESH, bool COMPACT, bool TAB>
__global__ void __launch_bounds__(1024, 1) iso_gather_rows_wide(const __grid_constant__ LaunchDev L)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    gather_rows_body<W, DEPTH, NU, MESH, COMPACT, TAB>(L, smem_raw, true, blockIdx.x, gridDim.x, blockDim.x);
}

// Sender-side form of an allgather phase.  In the prefix-trie schedule (Section III-B) a node's
// block is copied to every child node, and the children of one node live at different
// processes (one step along the phase's dimension per distinct coordinate).  Run as a gather,
// every child loads the parent block again - two loads of the same bytes within a few hundred
// nanoseconds for a Moore neighbourhood, both of which went to device memory.  Here a thread
// owns a unit position of the PARENT blocks of a process: it loads the unit once, from its
// own process (consecutive rows: a plain streaming read), and stores it to up to four
// destinations, each in the buffer of the process c steps further along the dimension
// (wrap-around by the row's coordinate).  Same CTA shape, row assignment and cp.async ring
// as the gather above; 16-byte units only.
struct alignas(16) FanDev {
    long long src_term;     // byte offset of the unit in the own source buffer
    long long dst_term[4];  // destination offset + c * rank stride * destination stride (no wrap)
    int32_t c[4];           // shift of destination e along the launch's dimension, in [0, p)
    uint8_t src_buf, n_dst;
    uint8_t dst_buf[4];
    uint8_t pad[2];
};
static_assert(sizeof(FanDev) == 64, "fan descriptors are read as four 16-byte words");

template <int DEPTH>
__global__ void __launch_bounds__(1024, 1) iso_fan_rows(const __grid_constant__ LaunchDev L)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    uint4 *const ring = reinterpret_cast<uint4 *>(smem_raw) + threadIdx.x;
    uint4 *const ring_end = ring + DEPTH * blockDim.x;
    const uint32_t CU = L.chunk_units, U = L.units_per_proc;
    const int G = (int)L.rows_per_pass;
    const int g = (int)(threadIdx.x / CU);
    const uint32_t ul = threadIdx.x - (uint32_t)g * CU;
    const long long r0 = L.row_lo + (long long)G * blockIdx.x + g;
    const bool active = g < G && r0 < L.row_hi && ul < U;
    const FanDev *table = reinterpret_cast<const FanDev *>(L.units);
    uint4 q0 = make_uint4(0, 0, 0, 0), q1 = q0, q2 = q0, q3 = q0;
    if (active) {
        const uint4 *raw = reinterpret_cast<const uint4 *>(table + ul);
        q0 = __ldg(raw); q1 = __ldg(raw + 1); q2 = __ldg(raw + 2); q3 = __ldg(raw + 3);
    }
    grid_dependency_wait();
    grid_launch_dependents();
    if (!active) return;
    const long long rstep = (long long)G * gridDim.x;
    const long long r_end = L.row_hi;
    const int p = (int)L.used_size[0];
    const long long wrap_ranks = (long long)L.used_wrap[0];

    for (uint32_t u = ul; u < U; u += CU) {
        if (u != ul) {
            const uint4 *raw = reinterpret_cast<const uint4 *>(table + u);
            q0 = __ldg(raw); q1 = __ldg(raw + 1); q2 = __ldg(raw + 2); q3 = __ldg(raw + 3);
        }
        const long long src_term = (long long)(((unsigned long long)q0.y << 32) | q0.x);
        const long long dt0 = (long long)(((unsigned long long)q0.w << 32) | q0.z);
        const long long dt1 = (long long)(((unsigned long long)q1.y << 32) | q1.x);
        const long long dt2 = (long long)(((unsigned long long)q1.w << 32) | q1.z);
        const long long dt3 = (long long)(((unsigned long long)q2.y << 32) | q2.x);
        const int sb = q3.z & 0xff, n_dst = (q3.z >> 8) & 0xff;
        const int db0 = (q3.z >> 16) & 0xff, db1 = q3.z >> 24, db2 = q3.w & 0xff, db3 = (q3.w >> 8) & 0xff;
        // a destination wraps around when the row's coordinate is at least p - c
        const int th0 = p - (int)q2.z, th1 = p - (int)q2.w, th2 = p - (int)q3.x, th3 = p - (int)q3.y;
        const long long stride_s = L.buf_stride[sb];
        unsigned char *const B0 = L.buf[db0] + dt0, *const B1 = L.buf[db1] + dt1;
        unsigned char *const B2 = L.buf[db2] + dt2, *const B3 = L.buf[db3] + dt3;
        const long long s0 = L.buf_stride[db0], s1 = L.buf_stride[db1], s2 = L.buf_stride[db2], s3 = L.buf_stride[db3];
        const long long src_step = rstep * stride_s;

        long long r_ld = r0;
        const unsigned char *src_ld = L.buf[sb] + src_term + r0 * stride_s;
#pragma unroll
        for (int i = 0; i < DEPTH; ++i) {
            if (r_ld < r_end) {
                cp_async<16>(ring + i * blockDim.x, src_ld);
                r_ld += rstep;
                src_ld += src_step;
            }
            cp_async_commit();
        }
        uint4 *slot = ring;
        for (long long r = r0; r < r_end; r += rstep) {
            cp_async_wait<DEPTH - 1>();
            const uint4 v = *slot;
            const uint32_t t = fastdiv(L.div_rstride[0], (uint32_t)r);
            const int x = (int)(t - fastdiv(L.div_size[0], t) * L.used_size[0]);
            *reinterpret_cast<uint4 *>(B0 + (r - (x >= th0 ? wrap_ranks : 0)) * s0) = v;
            if (n_dst > 1) *reinterpret_cast<uint4 *>(B1 + (r - (x >= th1 ? wrap_ranks : 0)) * s1) = v;
            if (n_dst > 2) *reinterpret_cast<uint4 *>(B2 + (r - (x >= th2 ? wrap_ranks : 0)) * s2) = v;
            if (n_dst > 3) *reinterpret_cast<uint4 *>(B3 + (r - (x >= th3 ? wrap_ranks : 0)) * s3) = v;
            if (r_ld < r_end) {
                cp_async<16>(slot, src_ld);
                r_ld += rstep;
                src_ld += src_step;
            }
            cp_async_commit();
            slot += blockDim.x;
            if (slot == ring_end) slot = ring;
        }
        cp_async_wait<0>();
    }
}

// All phases of a schedule in ONE cooperative launch: the CTAs run phase after phase and
// meet at a grid-wide barrier in between, which removes the launch ramp and drain of the
// per-phase kernels.  Every launch of the schedule must be a 16-byte vector launch on
// periodic dimensions.  The launch descriptors live in device memory and are copied to
// shared memory phase by phase.
struct MultiDev {
    const LaunchDev *launches;
    int n;
    unsigned long long *counter;  // arrivals at the grid barrier, never reset
    unsigned long long epoch;     // value of the counter when this launch began
    int *err;                     // set to 2 when a barrier wait gives up
    uint32_t max_polls;           // polls of one wait before it gives up
    uint32_t arrivals;            // arrivals that complete one barrier (the grid size, unless a test skews it)
};

constexpr uint32_t kBarrierPolls = 1u << 22;  // default poll limit of the waits on other CTAs

// Grid-wide barrier for a cooperative launch (all CTAs are resident).  One thread per CTA
// publishes the CTA's writes, counts itself in and polls the counter a bounded number of
// times; on expiry it raises the error flag and every thread of the CTA gets `false`.
__device__ __forceinline__ bool grid_barrier(const MultiDev &M, unsigned long long target, int *s_ok)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(M.counter, 1ULL);
        bool ok = true;
        uint32_t polls = 0;
        for (;;) {
            unsigned long long seen;
            asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(seen) : "l"(M.counter) : "memory");
            if (seen >= target) break;
            if (++polls >= M.max_polls) {
                ok = false;
                break;
            }
            __nanosleep(40);
        }
        __threadfence();
        if (!ok) atomicExch(M.err, 2);
        *s_ok = ok ? 1 : 0;
    }
    __syncthreads();
    return *s_ok != 0;
}

template <int DEPTH>
__global__ void __launch_bounds__(1024, 1) iso_gather_rows_multi(const __grid_constant__ MultiDev M)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ int s_ok;
    LaunchDev *sL = reinterpret_cast<LaunchDev *>(smem_raw);
    unsigned char *ring = smem_raw + ((sizeof(LaunchDev) + 127) / 128) * 128;
    for (int ph = 0; ph < M.n; ++ph) {
        const uint32_t *src = reinterpret_cast<const uint32_t *>(M.launches + ph);
        uint32_t *dst = reinterpret_cast<uint32_t *>(sL);
        for (uint32_t i = threadIdx.x; i < sizeof(LaunchDev) / 4; i += blockDim.x) dst[i] = __ldg(src + i);
        __syncthreads();
        switch (sL->n_used) {
        case 0: gather_rows_body<16, DEPTH, 0, false, false>(*sL, ring, false, blockIdx.x, gridDim.x, blockDim.x); break;
        case 1: gather_rows_body<16, DEPTH, 1, false, false>(*sL, ring, false, blockIdx.x, gridDim.x, blockDim.x); break;
        case 2: gather_rows_body<16, DEPTH, 2, false, false>(*sL, ring, false, blockIdx.x, gridDim.x, blockDim.x); break;
        case 3: gather_rows_body<16, DEPTH, 3, false, false>(*sL, ring, false, blockIdx.x, gridDim.x, blockDim.x); break;
        default: gather_rows_body<16, DEPTH, ISO_MAX_DIMS, false, false>(*sL, ring, false, blockIdx.x, gridDim.x, blockDim.x); break;
        }
        if (ph + 1 < M.n && !grid_barrier(M, M.epoch + (unsigned long long)(ph + 1) * M.arrivals, &s_ok)) return;
    }
}

// Pipelined one-launch execution.  The torus is cut into slabs of planes of dimension 0
// and the work into items (slab, launch of the schedule); all CTAs go through the items in
// one fixed order, each taking its share of an item's rows.  Instead of a grid barrier
// between phases, every item has a counter of the CTAs that have finished it, and a CTA
// starts item i once the item it depends on (the slab's previous phase, or the last reader
// of the intermediate place it overwrites) has been finished by all CTAs.  The order puts
// other items in between, so that wait is normally over before it begins, and a slab's
// intermediate blocks are read back a few items after they were written, out of L2.
struct WaveItem {
    int wait_item;        // item that must be complete first (-1: none)
    uint32_t cta_offset;  // rotation of the CTA numbering, continues the round robin of the item before
    int variant;          // 0..4: dense descriptors with 0, 1, 2, 3, any shifted dimensions; 5..8: compact with 1, 2, 3, any
    int pad;
};

struct WaveDev {
    const LaunchDev *launches;  // one complete descriptor per item (row range and buffers set)
    const WaveItem *items;
    int n;
    unsigned long long *done;   // per item: arrivals of CTAs, never reset
    unsigned long long target;  // arrivals that mean "complete" for this start
    int *err;                   // set to 2 when a wait gives up
    uint32_t max_polls;         // polls of one wait before it gives up
};

template <int DEPTH>
__global__ void __launch_bounds__(1024, 1) iso_gather_rows_wave(const __grid_constant__ WaveDev M)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ int s_ok;
    __shared__ WaveItem s_item;
    LaunchDev *sL = reinterpret_cast<LaunchDev *>(smem_raw);
    unsigned char *ring = smem_raw + ((sizeof(LaunchDev) + 127) / 128) * 128;
    for (int i = 0; i < M.n; ++i) {
        const uint32_t *src = reinterpret_cast<const uint32_t *>(M.launches + i);
        uint32_t *dst = reinterpret_cast<uint32_t *>(sL);
        for (uint32_t k = threadIdx.x; k < sizeof(LaunchDev) / 4; k += blockDim.x) dst[k] = __ldg(src + k);
        if (threadIdx.x == 0) {
            const WaveItem it = M.items[i];
            s_item = it;
            bool ok = true;
            if (it.wait_item >= 0) {
                const unsigned long long *flag = M.done + it.wait_item;
                uint32_t polls = 0;
                for (;;) {
                    unsigned long long seen;
                    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(seen) : "l"(flag) : "memory");
                    if (seen >= M.target) break;
                    if (++polls >= M.max_polls) {
                        ok = false;
                        break;
                    }
                    __nanosleep(32);
                }
                if (!ok) atomicExch(M.err, 2);
            }
            s_ok = ok ? 1 : 0;
        }
        __syncthreads();
        if (!s_ok) return;
        const uint32_t n_cta = gridDim.x;
        uint32_t cta = blockIdx.x + n_cta - s_item.cta_offset;
        if (cta >= n_cta) cta -= n_cta;
        switch (s_item.variant) {
        case 0: gather_rows_body<16, DEPTH, 0, false, false>(*sL, ring, false, cta, n_cta, blockDim.x); break;
        case 1: gather_rows_body<16, DEPTH, 1, false, false>(*sL, ring, false, cta, n_cta, blockDim.x); break;
        case 2: gather_rows_body<16, DEPTH, 2, false, false>(*sL, ring, false, cta, n_cta, blockDim.x); break;
        case 3: gather_rows_body<16, DEPTH, 3, false, false>(*sL, ring, false, cta, n_cta, blockDim.x); break;
        case 4: gather_rows_body<16, DEPTH, ISO_MAX_DIMS, false, false>(*sL, ring, false, cta, n_cta, blockDim.x); break;
        case 5: gather_rows_body<16, DEPTH, 1, false, true>(*sL, ring, false, cta, n_cta, blockDim.x); break;
        case 6: gather_rows_body<16, DEPTH, 2, false, true>(*sL, ring, false, cta, n_cta, blockDim.x); break;
        case 7: gather_rows_body<16, DEPTH, 3, false, true>(*sL, ring, false, cta, n_cta, blockDim.x); break;
        default: gather_rows_body<16, DEPTH, ISO_MAX_DIMS, false, true>(*sL, ring, false, cta, n_cta, blockDim.x); break;
        }
        // all stores of this CTA for the item are issued: publish them and count the CTA in
        __syncthreads();
        if (threadIdx.x == 0) {
            __threadfence();
            atomicAdd(M.done + i, 1ULL);
        }
    }
}

// Same ownership scheme with the data held in registers, for 1- and 2-byte units (cp.async
// moves at least 4 bytes): UNROLL independent loads in flight before the first store.
template <int W, int UNROLL>
__global__ void __launch_bounds__(256) iso_gather_rows_reg(const __grid_constant__ LaunchDev L)
{
    using V = typename VecOf<W>::type;
    const uint32_t CU = L.chunk_units, U = L.units_per_proc;
    const int G = (int)L.rows_per_pass;
    const int g = (int)(threadIdx.x / CU);
    const uint32_t ul = threadIdx.x - (uint32_t)g * CU;
    grid_dependency_wait();
    grid_launch_dependents();
    const long long r0 = L.row_lo + (long long)G * blockIdx.x + g;
    if (g >= G || r0 >= L.row_hi) return;
    const long long rstep = (long long)G * gridDim.x;

    for (uint32_t u = ul; u < U; u += CU) {
        const UnitRegs R = load_unit(L, u);
        for (long long rb = r0; rb < L.row_hi; rb += rstep * UNROLL) {
            V val[UNROLL];
            V *dst[UNROLL];
#pragma unroll
            for (int k = 0; k < UNROLL; ++k) {
                const long long r = rb + k * rstep;
                dst[k] = nullptr;
                if (r < L.row_hi) {
                    long long wrap = 0;
                    bool valid = true;
                    for (int e = 0; e < L.n_used; ++e) {
                        const uint32_t t = fastdiv(L.div_rstride[e], (uint32_t)r);
                        const int x = (int)(t - fastdiv(L.div_size[e], t) * L.used_size[e]);
                        if ((L.mesh_mask >> e) & 1) {
                            const int y = x - R.c[e];
                            valid = valid && y >= 0 && y < (int)L.used_size[e];
                        } else if (x < R.c[e]) {
                            wrap += L.used_wrap[e];
                        }
                    }
                    if (valid) {
                        val[k] = *reinterpret_cast<const V *>(R.A + (r + wrap) * R.stride_s);
                        dst[k] = reinterpret_cast<V *>(R.B + r * R.stride_d);
                    }
                }
            }
#pragma unroll
            for (int k = 0; k < UNROLL; ++k)
                if (dst[k]) *dst[k] = val[k];
        }
    }
}

// Does nothing: a chain of these measures what a kernel launch costs on the stream
// (with and without programmatic dependent launch), the floor under every short phase.
__global__ void iso_empty_kernel(int)
{
    grid_dependency_wait();
    grid_launch_dependents();
}

// ---- asynchronous bulk copies (TMA, untiled form) ------------------------------------

__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// global -> shared, completion reported on an mbarrier of this CTA
__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gsrc, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

// shared -> global, tracked by the thread's bulk async-group
__device__ __forceinline__ void bulk_store(void *gdst, const void *smem_src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_addr(smem_src)),
                 "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Upper bound on polls of one mbarrier before the kernel gives up and reports an error.
constexpr uint32_t kBulkWaitPolls = 1u << 22;

// Bulk gather for large parts: every thread drives its own two-stage pipeline of chunks,
//   global --cp.async.bulk--> shared (mbarrier) --cp.async.bulk--> global (bulk group),
// so that per thread one load and one store are in flight at any time and the data never
// passes through registers.  All addresses and sizes are multiples of 16 bytes.
__global__ void __launch_bounds__(256) iso_gather_bulk(const __grid_constant__ LaunchDev L)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint32_t chunk = L.width;
    unsigned char *s_data = smem_raw;                                                           // threads * 2 * chunk
    uint64_t *s_bar = reinterpret_cast<uint64_t *>(smem_raw + (size_t)blockDim.x * 2 * chunk);  // threads * 2
    uint32_t *s_coord =
        reinterpret_cast<uint32_t *>(smem_raw + (size_t)blockDim.x * 2 * chunk + (size_t)blockDim.x * 16);

    const long long r0 = L.row_lo + (long long)blockIdx.x * L.tile_procs;
    const long long left = L.row_hi - r0;
    const int np = left <= 0 ? 0 : (int)(left < L.tile_procs ? left : L.tile_procs);
    tile_coordinates(L, r0, np, s_coord);
    uint64_t *bar = s_bar + 2 * threadIdx.x;
    unsigned char *stage = s_data + (size_t)threadIdx.x * 2 * chunk;
    mbar_init(&bar[0], 1);
    mbar_init(&bar[1], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
    __syncthreads();
    grid_dependency_wait();
    grid_launch_dependents();

    const uint32_t total = (uint32_t)np * L.units_per_proc;
    const uint32_t n = threadIdx.x < total ? (total - threadIdx.x + blockDim.x - 1) / blockDim.x : 0;
    uint32_t parity_bits = 0;   // bit s: parity the next wait on stage s has to see
    uint32_t pending_bits = 0;  // bit s: a load into stage s has been issued and not yet awaited
    bool failed = false;

    auto await = [&](uint32_t s) {
        uint32_t polls = 0;
        while (!mbar_try_wait(&bar[s], (parity_bits >> s) & 1u)) {
            if (++polls >= kBulkWaitPolls) {
                failed = true;
                return;
            }
        }
        parity_bits ^= 1u << s;
        pending_bits &= ~(1u << s);
    };

    UnitAddr cur{}, nxt{};
    if (n > 0) {
        cur = decode_unit(L, r0, threadIdx.x, s_coord);
        if (cur.valid) {
            mbar_expect_tx(&bar[0], cur.bytes);
            bulk_load(stage, cur.src, cur.bytes, &bar[0]);
            pending_bits |= 1u;
        }
    }
    for (uint32_t k = 0; k < n; ++k) {
        const uint32_t s = k & 1u;
        if (k + 1 < n) {
            bulk_wait_read_all();  // the other stage was last read by the store of item k-1
            nxt = decode_unit(L, r0, threadIdx.x + (k + 1) * blockDim.x, s_coord);
            if (nxt.valid && !failed) {
                mbar_expect_tx(&bar[s ^ 1u], nxt.bytes);
                bulk_load(stage + (size_t)(s ^ 1u) * chunk, nxt.src, nxt.bytes, &bar[s ^ 1u]);
                pending_bits |= 1u << (s ^ 1u);
            }
        }
        if (cur.valid && !failed) {
            await(s);
            if (!failed) {
                fence_async_smem();
                bulk_store(cur.dst, stage + (size_t)s * chunk, cur.bytes);
                bulk_commit();
            }
        }
        cur = nxt;
    }
    // on the error path a load may still be in flight: give it one more bounded wait so that
    // it does not land in shared memory that has been handed to another CTA
    for (uint32_t s = 0; s < 2; ++s)
        if (pending_bits >> s & 1u) {
            bool keep = failed;
            failed = false;
            await(s);
            failed = failed || keep;
        }
    bulk_wait_all();
    if (failed) atomicExch(L.err, 1);
}

// Chunk `u` of the long pieces of row r (the bulk side of a hybrid launch): like decode_unit,
// with the row's coordinates computed on the spot instead of read from a tile's table.
__device__ __forceinline__ UnitAddr decode_row_unit(const LaunchDev &L, long long r, uint32_t u)
{
    uint32_t t;
    if (L.uniform_units) {
        t = fastdiv(L.div_uniform, u);
    } else {
        t = L.lookup[u >> L.lookup_shift];
        while (t + 1 < L.nparts && __ldg(&L.parts[t + 1].first_unit) <= u) ++t;
    }
    const PartDev *p = L.parts + t;
    const uint32_t k = u - __ldg(&p->first_unit);
    long long rs = r + __ldg(&p->rank_delta);
    const int nnz = __ldg(&p->nnz);
    for (int e = 0; e < nnz; ++e) {
        const int dk = __ldg(&p->dim[e]);
        const int c = __ldg(&p->c[e]);
        const uint32_t q = fastdiv(L.div_rstride[dk], (uint32_t)r);
        const int x = (int)(q - fastdiv(L.div_size[dk], q) * L.used_size[dk]);
        if (x < c) rs += (long long)L.used_size[dk] * L.used_rstride[dk];
    }
    const long long within = (long long)k * L.width;
    const long long rest = __ldg(&p->len) - within;
    UnitAddr a;
    a.src = L.buf[__ldg(&p->src_buf)] + rs * L.buf_stride[__ldg(&p->src_buf)] + __ldg(&p->src_off) + within;
    a.dst = L.buf[__ldg(&p->dst_buf)] + r * L.buf_stride[__ldg(&p->dst_buf)] + __ldg(&p->dst_off) + within;
    a.bytes = (uint32_t)(rest < (long long)L.width ? rest : (long long)L.width);
    a.valid = true;
    return a;
}

// Ragged rows (irregular collectives): the vector gather and the bulk gather in ONE kernel.
// A row of such a collective is a few long blocks between many short pieces.  Moved unit by
// unit, the long blocks make up most of the 16-byte units, and every unit costs a cp.async,
// a shared-memory load and a store through the same load/store queue, whose capacity, not
// memory bandwidth, then bounds the kernel.  Here the first warps run the vector gather over
// the short pieces and ragged ends only, while the last warps (S.chunk_units threads) move the
// long 16-byte-aligned bodies of the SAME rows (same assignment of row groups to CTAs) with
// bulk copies, global -> shared -> global, two stages per lane, as iso_gather_bulk does: the bulk
// copies have their own queue, so both engines work at the same time, and pieces that share
// a 32-byte sector with a long body still move within a few rows of it.  Periodic
// dimensions only.  L: the vector side; S: the bulk side (same row range).
template <int DEPTH, int NU, bool TAB>
__global__ void __launch_bounds__(1024, 1) iso_gather_rows_hybrid(const __grid_constant__ LaunchDev L,
                                                                  const __grid_constant__ LaunchDev S)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint32_t lanes = S.chunk_units;  // threads of the bulk warps
    const uint32_t nvec = blockDim.x - lanes;
    if (threadIdx.x < nvec) {
        gather_rows_body<0, DEPTH, NU, false, false, TAB>(L, smem_raw, true, blockIdx.x, gridDim.x, nvec);
        return;
    }
    const uint32_t lane = threadIdx.x - nvec;
    const uint32_t chunk = S.width;
    unsigned char *stage = smem_raw + S.side_offset + (size_t)lane * 2 * chunk;
    uint64_t *bar = reinterpret_cast<uint64_t *>(smem_raw + S.side_offset + (size_t)lanes * 2 * chunk) + 2 * lane;
    mbar_init(&bar[0], 1);
    mbar_init(&bar[1], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
    __syncwarp();
    if (TAB) __syncthreads();  // the barrier the vector warps pass after filling their coordinate table
    grid_dependency_wait();
    grid_launch_dependents();

    // items of this CTA: (row group it, row slot g, chunk u), consecutive lanes on consecutive chunks
    const uint32_t G = L.rows_per_pass, U = S.units_per_proc;
    const long long group0 = S.row_lo + (long long)G * blockIdx.x;
    const long long rstep = (long long)G * gridDim.x;
    const uint32_t per_group = G * U;
    uint32_t total = 0;
    if (group0 < S.row_hi) total = (uint32_t)((S.row_hi - group0 + rstep - 1) / rstep) * per_group;
    uint32_t parity_bits = 0, pending_bits = 0;
    bool failed = false;
    auto await = [&](uint32_t s) {
        uint32_t polls = 0;
        while (!mbar_try_wait(&bar[s], (parity_bits >> s) & 1u)) {
            if (++polls >= kBulkWaitPolls) {
                failed = true;
                return;
            }
        }
        parity_bits ^= 1u << s;
        pending_bits &= ~(1u << s);
    };
    auto item = [&](uint32_t k) -> UnitAddr {
        const uint32_t it = k / per_group, rem = k - it * per_group;
        const uint32_t g = rem / U, u = rem - g * U;
        const long long r = group0 + (long long)it * rstep + g;
        UnitAddr a{};
        a.valid = false;
        if (r < S.row_hi) a = decode_row_unit(S, r, u);
        return a;
    };

    UnitAddr cur{}, nxt{};
    cur.valid = nxt.valid = false;
    uint32_t s = 0;  // stage of `cur`
    if (lane < total) {
        cur = item(lane);
        if (cur.valid) {
            mbar_expect_tx(&bar[0], cur.bytes);
            bulk_load(stage, cur.src, cur.bytes, &bar[0]);
            pending_bits |= 1u;
        }
    }
    for (uint32_t k = lane; k < total; k += lanes) {
        nxt.valid = false;
        if (k + lanes < total) {
            bulk_wait_read_all();  // the other stage was last read by the store of the item before
            nxt = item(k + lanes);
            if (nxt.valid && !failed) {
                mbar_expect_tx(&bar[s ^ 1u], nxt.bytes);
                bulk_load(stage + (size_t)(s ^ 1u) * chunk, nxt.src, nxt.bytes, &bar[s ^ 1u]);
                pending_bits |= 1u << (s ^ 1u);
            }
        }
        if (cur.valid && !failed) {
            await(s);
            if (!failed) {
                fence_async_smem();
                bulk_store(cur.dst, stage + (size_t)s * chunk, cur.bytes);
                bulk_commit();
            }
        }
        cur = nxt;
        s ^= 1u;
    }
    // on the error path a load may still be in flight: one more bounded wait, so that it does
    // not land in shared memory that has been handed to another CTA
    for (uint32_t q = 0; q < 2; ++q)
        if (pending_bits >> q & 1u) {
            const bool keep = failed;
            failed = false;
            await(q);
            failed = failed || keep;
        }
    bulk_wait_all();
    if (failed) atomicExch(S.err, 1);
}

}  // namespace iso
