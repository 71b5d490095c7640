// Internal host-side types of the isomorphic neighbourhood collectives library.
#pragma once

#include <cstdint>
#include <vector>

#include "iso.h"

namespace iso {

struct Comm {
    int refcount = 1;
    int d = 0;
    int s = 0;
    int dims[ISO_MAX_DIMS] = {0};
    int periodic[ISO_MAX_DIMS] = {0};
    int64_t P = 1;
    int64_t rank_stride[ISO_MAX_DIMS] = {0};  // ranks between neighbours along dimension j
    std::vector<int> coords;                  // s*d, as given by the caller
};

// One line of the executed schedule, before it is lowered to kernel launches.
struct Part {
    int phase = 0;
    int round = -1;
    int slot = 0;
    int src_buf = ISO_BUF_SEND;
    int dst_buf = ISO_BUF_RECV;
    int64_t src_off = 0;
    int64_t dst_off = 0;
    int64_t len = 0;
    int shift[ISO_MAX_DIMS] = {0};  // residue in [0,p_j) for periodic dimensions, signed for mesh ones
    int check[ISO_MAX_DIMS] = {0};  // mesh dimensions: process x takes part only if 0 <= x_j - check_j < p_j
};

// Exact unsigned 32-bit division by an invariant divisor (Granlund & Montgomery 1994,
// round-up method): q = (t + ((n - t) >> s1)) >> s2 with t = mulhi(m, n).
struct FastDiv {
    uint32_t m = 1, s1 = 0, s2 = 0, div = 1;
};
FastDiv make_fastdiv(uint32_t divisor);
inline uint32_t fastdiv_host(const FastDiv &f, uint32_t n)
{
    uint32_t t = (uint32_t)(((uint64_t)f.m * n) >> 32);
    return (t + ((n - t) >> f.s1)) >> f.s2;
}

// A part as one kernel launch sees it (after splitting into aligned pieces).
struct LoweredPart {
    Part p;            // offsets / len of this piece
    uint32_t first_unit = 0;
    uint32_t units = 0;
    int width = 16;    // bytes per unit of this piece (differs between pieces in a launch of mixed widths)
};

enum { KERNEL_VEC = 0, KERNEL_BULK = 1, KERNEL_FAN = 2 };

// Sender-side form of an allgather phase (Section III-B: a trie edge carries one block once):
// a parent block, read once from the process that holds it, and the places it is copied to.
struct FanDst {
    int buf = ISO_BUF_RECV;
    int64_t off = 0;
    int c = 0;  // the destination process is the source process shifted by +c along the phase's dimension, c in [0, p)
};
struct FanParent {
    int src_buf = ISO_BUF_SEND;
    int64_t src_off = 0;
    int64_t len = 0;
    std::vector<FanDst> dsts;  // at most kFanDsts
};
constexpr int kFanDsts = 4;  // destinations per descriptor; a parent with more is listed several times
constexpr int64_t kHybridMinBytes = 256;  // 16-byte-aligned pieces of a ragged row from which bulk copies take over
constexpr int kMaxOwnSlabs = 128;          // most slabs of dimension 0 the library chooses by itself
constexpr double kSlabLaunchBytes = 52e6;  // what one launch of a slab may write so that it and its reader share the L2
constexpr int kMaxVecUnits = 8192;  // unit positions per process in one vector launch
constexpr int kVecDepth = 8;        // cp.async ring slots per thread in the vector kernel
constexpr int kWideDepth = 12;      // the same in CTAs of more than 256 threads (one CTA per SM)
constexpr int kHybridDepth = 6;     // the same for the vector warps of a hybrid launch (most of the shared memory stages bulk copies)
constexpr size_t kHybridStageBytes = 128 * 1024;  // staging area of the bulk warps of a hybrid launch

struct LaunchPlan {
    int kernel = KERNEL_VEC;
    int width = 16;       // bytes per unit (vector kernel; 0: mixed, every piece has its own); chunk bytes (bulk kernel)
    int phase = 0;
    std::vector<LoweredPart> parts;
    uint32_t units_per_proc = 0;
    uint32_t uniform_units = 0;  // >0: every part has this many units
    int lookup_shift = 0;
    std::vector<uint16_t> lookup;  // unit >> lookup_shift -> index of the part holding that unit
    uint32_t chunk_units = 1;    // vector kernel: unit positions per row slot
    uint32_t rows_per_pass = 1;  // vector kernel: rows a CTA handles at the same time
    int tile_procs = 1;
    int threads = 256;
    int64_t grid = 0;
    size_t smem = 0;
    int n_used = 0;
    int used_dim[ISO_MAX_DIMS] = {0};
    int max_nnz = 0;       // most dimensions any one part shifts along
    bool compact = false;  // vector kernel: unit descriptors list only the shifted dimensions
    int64_t rows_hint = 0; // vector kernel: rows the grid holds at a time when CTAs cover whole rows (slab heuristic)
    int col_split = 1;     // vector kernel: column chunks of a row longer than a CTA, one CTA per chunk and row (1: none)
    std::vector<LaunchPlan> side;  // mixed-width vector launch: at most one bulk-copy plan for the long bodies of its rows,
                                   // run by one extra warp of the same CTAs
    std::vector<FanParent> fans;  // KERNEL_FAN: the launch as parents and their destinations (parts: the same copies, one per destination)
    // byte offsets of this launch's tables inside the request's device blob
    size_t parts_off = 0, lookup_off = 0, units_off = 0;
};

// Experiment knobs, read from the environment ONCE, when a request is created, so that a
// persistent request keeps one plan however the environment changes between its starts.
// -1 (or 0 where stated) means "not set": the library's own choice applies.
struct Knobs {
    int pack_by_round = -1;   // ISO_PACK_BY_ROUND: intermediate places grouped by reading round (0/1)
    int lazy_final = -1;      // ISO_LAZY_FINAL: postpone every final hop to the last phase (0/1)
    int mixed = -1;           // ISO_MIXED: 0 = one launch per unit width instead of one of mixed widths
    int64_t bulk_chunk = 0;   // ISO_BULK_CHUNK: chunk bytes of the bulk kernel (0: automatic)
    int vec_threads = 0;      // ISO_VEC_THREADS: 256 or 512 for narrower CTAs (0: up to 1024)
    int vec_ctas_per_sm = 0;  // ISO_VEC_CTAS_PER_SM: CTAs per SM of the 256-thread shapes (0: automatic)
    int64_t bulk_tile = 0;    // ISO_BULK_TILE: processes per CTA of the bulk kernel (0: automatic)
    int host_slabs = -1;      // ISO_HOST_SLABS: slabs of the pipelined host-buffer path (-1: automatic)
    int graph = -1;           // ISO_GRAPH: graph replay on/off
    int slabs = -1;           // ISO_SLABS: slab count of Iso_Start
    int chains = -1;          // ISO_CHAINS
    bool no_pdl = false;      // ISO_NO_PDL: plain launches instead of programmatic dependent ones
    bool tune_log = false;    // ISO_TUNE_LOG: the tuner prints every plan it times
    int sender_side = -1;     // ISO_SENDER_SIDE: 0 never, 1 automatic, 2 wherever possible (allgather phases; -1: the request's setting)
    int hybrid = -1;          // ISO_HYBRID: 1 = long bodies of ragged rows through bulk warps, 0 = not (-1: the request's setting)
    bool col_split = true;    // ISO_COL_SPLIT=0: rows longer than a CTA are covered in passes instead of column chunks
    bool host_graph = true;   // ISO_HOST_GRAPH=0: the pipelined host-buffer path is never replayed from a graph
    bool coord_table = true;  // ISO_COORD_TABLE=0: row coordinates by division in every thread
    bool l2_keep = true;      // ISO_L2_KEEP=0: no eviction-priority hint on stores into the intermediate buffer
    int ag_order = -1;        // ISO_AG_ORDER=0/1: allgather visits the dimensions first-to-last / last-to-first
};
Knobs read_knobs();

struct Request {
    Comm *comm = nullptr;
    Knobs knobs;
    int kind = ISO_KIND_ALLTOALL;
    int alg = ISO_ALG_COMBINING;
    int fusion = 1;
    int dim_order[ISO_MAX_DIMS] = {0, 1, 2, 3, 4, 5, 6, 7};  // allgather: dimension visited k-th (Section III-B)
    int64_t bulk_threshold = 512;        // in force (set by lower_schedule)
    int64_t bulk_threshold_asked = -1;   // Iso_request_set_bulk_threshold; -1: chosen by the library
    int layout = ISO_LAYOUT_PACKED;
    int slab_request = 0;     // slabs of dimension 0 Iso_Start runs one after the other (0: automatic, 1: none)
    bool persistent = false;  // run all phases in one cooperative launch when the schedule allows
    const unsigned char *send = nullptr;
    unsigned char *recv = nullptr;
    int s = 0;
    std::vector<int64_t> len, sdispl, rdispl;
    int64_t send_stride = 0, recv_stride = 0, inter_stride = 0;
    std::vector<Part> parts;           // schedule in execution order
    std::vector<LaunchPlan> launches;  // lowered schedule
    Iso_stats stats{};
    // device side (owned by iso_api.cu)
    bool dirty = true;
    void *d_blob = nullptr;
    unsigned char *d_inter = nullptr;        // first usable byte (behind the leading guard band)
    unsigned char *d_inter_alloc = nullptr;  // the allocation: guard band, buffer, guard band
    int64_t d_inter_bytes = 0;
    int *d_err = nullptr;
    unsigned long long *d_counter = nullptr;  // grid-barrier arrivals (one-launch execution)
    unsigned long long epoch = 0;             // counter value at the next launch
    int multi_grid = 0;                       // > 0: one-launch execution with this grid
    size_t multi_smem = 0, multi_launches_off = 0;
    int *h_err = nullptr;
    void *last_stream = nullptr;
    bool started = false;
    std::vector<std::pair<long long, long long>> slab_plan;  // row ranges of the slabs (empty: whole torus at once)
    int64_t inter_rows = 0;            // processes the intermediate buffer holds
    std::vector<void *> host_streams;  // pipelined host-buffer path: two upload and two download streams
    std::vector<void *> slab_events;   // its events
    void *host_main_stream = nullptr;  // origin stream when that path is captured into a graph
    void *host_graph_exec = nullptr;   // cudaGraphExec_t of one pipelined host-buffer start
    const void *host_graph_hs = nullptr, *host_graph_hr = nullptr;  // the host buffers that graph copies from / to
    const void *host_last_hs = nullptr, *host_last_hr = nullptr;    // the host buffers of the last such start
    std::vector<void *> host_timing;   // timing events of its last call: uploads, downloads, whole call (begin, end each)
    bool host_timed = false;
    int host_slabs_used = 0;
    int sm_count = 148;  // a B200's; replaced by the current device's count before the first start
    int chains_request = 1;     // slabs to run side by side, as asked for
    bool graph_request = false; // graph replay, as asked for
    int chains = 1;             // slabs that run side by side (each on its share of the SMs)
    bool use_graph = false;     // Iso_Start replays a captured graph of the launches
    void *graph_exec = nullptr; // cudaGraphExec_t, built at the first Iso_Start after a change
    // pipelined one-launch execution (items = slab x launch, per-item completion counters)
    int wave_request = 0;       // 0: off, 1: one slab, n >= 2: n slabs of dimension 0
    bool wave_ok = false;       // the lowered schedule allows it (decided before the buffers are sized)
    int wave_slabs = 0;         // slabs in use (0: not in this mode)
    int wave_grid = 0;          // > 0: Iso_Start makes one cooperative launch of this many CTAs
    int wave_items = 0;
    size_t wave_smem = 0, wave_launches_off = 0, wave_items_off = 0;
    unsigned long long wave_run = 0;  // starts since the counters were last zeroed
    int wave_counters = 0;      // counters allocated in d_counter
    bool hybrid = false;        // launches of mixed widths hand their long bodies to bulk warps (Iso_request_set_hybrid)
    int sender_side = 1;        // allgather phases in sender-side form: 0 never, 1 where measured faster, 2 wherever possible
    uint32_t wait_limit = 1u << 22;  // polls before a device-side wait on other CTAs gives up
    int skew_next = 0;          // testing: extra arrivals the next cooperative start waits for (one shot)
};

// Builds r.parts, r.inter_stride and the schedule statistics from r.comm, r.kind, r.alg,
// r.fusion and the block layout.  Returns an ISO_* code.
// Default visiting order of the allgather's prefix trie for this neighbourhood (fills r.dim_order).
void default_dimension_order(Request &r);
int build_schedule(Request &r);

// Splits parts into aligned pieces, groups them into kernel launches and fills the launch
// geometry.  `send_addr` / `recv_addr` / `inter_addr` are only used for their alignment.
int lower_schedule(Request &r, uintptr_t send_addr, uintptr_t recv_addr, uintptr_t inter_addr);

// Checks the executed parts for hazards: every range inside its buffer, no write to the send
// buffer, and within a phase no written range overlapping another written or any read range.
int validate_schedule(const Request &r);

}  // namespace iso
