// Host-side schedule computation for the isomorphic neighbourhood collectives.
//
// The schedules are those of the paper "Message-Combining Algorithms for Isomorphic,
// Sparse Collective Communication":
//   * Section V    - message combining with direct communication along the dimensions:
//                    per dimension the neighbours are bucketed by their coordinate, one
//                    round per distinct non-zero coordinate, every block hops once per
//                    dimension in which its coordinate is non-zero;
//   * Algorithm 1  - the alternating buffer rule (receive into the user's receive buffer
//                    when an odd number of hops remains, else into the intermediate
//                    buffer) and the hop-by-hop torus schedule;
//   * Section III-B- the prefix trie of the allgather: a block is routed once per
//                    distinct prefix;
//   * Listing 3    - the straightforward schedule, every block straight from its source.
// Because all processes follow the same steps, a schedule is a process-independent list of
// parts "copy len bytes from (buffer, offset) of the process at -shift to (buffer, offset)
// of myself"; the kernels apply every part to every process.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <map>
#include <numeric>

#include "iso_internal.h"

namespace iso {

FastDiv make_fastdiv(uint32_t d)
{
    FastDiv f;
    f.div = d ? d : 1;
    d = f.div;
    uint32_t l = 0;
    while (l < 32 && ((uint64_t)1 << l) < d) ++l;  // l = ceil(log2 d)
    uint64_t two_l = (uint64_t)1 << l;
    f.m = (uint32_t)((((two_l - d) << 32) / d) + 1);
    f.s1 = l < 1 ? l : 1;
    f.s2 = l > 0 ? l - 1 : 0;
    return f;
}

Knobs read_knobs()
{
    Knobs k;
    auto num = [](const char *name, long long unset) -> long long {
        const char *v = std::getenv(name);
        return v ? std::atoll(v) : unset;
    };
    k.pack_by_round = (int)num("ISO_PACK_BY_ROUND", -1);
    k.lazy_final = (int)num("ISO_LAZY_FINAL", -1);
    k.mixed = (int)num("ISO_MIXED", -1);
    k.bulk_chunk = num("ISO_BULK_CHUNK", 0);
    k.vec_threads = (int)num("ISO_VEC_THREADS", 0);
    k.vec_ctas_per_sm = (int)num("ISO_VEC_CTAS_PER_SM", 0);
    k.bulk_tile = num("ISO_BULK_TILE", 0);
    k.host_slabs = (int)num("ISO_HOST_SLABS", -1);
    k.graph = (int)num("ISO_GRAPH", -1);
    k.slabs = (int)num("ISO_SLABS", -1);
    k.chains = (int)num("ISO_CHAINS", -1);
    k.no_pdl = num("ISO_NO_PDL", 0) != 0;
    k.tune_log = std::getenv("ISO_TUNE_LOG") != nullptr;
    k.sender_side = (int)num("ISO_SENDER_SIDE", -1);
    k.coord_table = num("ISO_COORD_TABLE", 1) != 0;
    k.host_graph = num("ISO_HOST_GRAPH", 1) != 0;
    k.hybrid = (int)num("ISO_HYBRID", -1);
    k.col_split = num("ISO_COL_SPLIT", 1) != 0;
    k.ag_order = num("ISO_AG_ORDER", -1);
    k.l2_keep = num("ISO_L2_KEEP", 1) != 0;
    return k;
}

namespace {

int reduce_mod(int c, int p)
{
    int x = c % p;
    return x < 0 ? x + p : x;
}

// representative of smallest magnitude, ties towards the positive one
int symmetric_rep(int residue, int p) { return 2 * (int64_t)residue <= p ? residue : residue - p; }

struct Geometry {
    int d, s;
    std::vector<int> red;  // s*d reduced coordinates
    const int *at(int i) const { return red.data() + (size_t)i * d; }
};

// Order of the rounds inside one dimension: positive coordinates by increasing
// magnitude, then negative ones by increasing magnitude (Algorithm 1 treats the positive
// coordinates first); keys of fused dimension groups are compared coordinate by coordinate.
struct RoundOrder {
    const int *dims;
    const int *periodic;  // on a mesh dimension the coordinates are signed and taken as they are
    int j0, j1;
    bool operator()(const std::vector<int> &a, const std::vector<int> &b) const
    {
        for (int j = j0; j < j1; ++j) {
            int sa = periodic[j] ? symmetric_rep(a[j - j0], dims[j]) : a[j - j0];
            int sb = periodic[j] ? symmetric_rep(b[j - j0], dims[j]) : b[j - j0];
            if (sa == sb) continue;
            bool na = sa < 0, nb = sb < 0;
            if (na != nb) return nb;  // non-negative first
            return std::abs(sa) < std::abs(sb);
        }
        return false;
    }
};

struct Groups {
    int n = 0;
    int begin[ISO_MAX_DIMS + 1] = {0};
};

Groups make_groups(int d, int fusion)
{
    Groups g;
    int width = fusion <= 1 ? 1 : fusion;
    for (int j = 0; j < d; j += width) g.begin[g.n++] = j;
    g.begin[g.n] = d;
    return g;
}

bool group_nonzero(const int *v, int j0, int j1)
{
    for (int j = j0; j < j1; ++j)
        if (v[j]) return true;
    return false;
}

int64_t round_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

void add_local_copy(Request &r, int slot, std::vector<Part> &out)
{
    Part p;
    p.phase = 0;
    p.round = -1;
    p.slot = slot;
    p.src_buf = ISO_BUF_SEND;
    p.dst_buf = ISO_BUF_RECV;
    p.src_off = r.sdispl[slot];
    p.dst_off = r.rdispl[slot];
    p.len = r.len[slot];
    out.push_back(p);
}

// --------------------------------------------------------------------------------------
// Listing 3, run as one pass: block i comes straight from the process at -C^i.
int build_direct(Request &r, const Geometry &g)
{
    const Comm &c = *r.comm;
    int locals = 0, parts = 0;
    for (int i = 0; i < g.s; ++i) {
        if (r.len[i] == 0) continue;
        const int *v = g.at(i);
        bool reachable = true, zero = true;
        for (int j = 0; j < g.d; ++j) {
            if (!c.periodic[j] && std::abs((int64_t)v[j]) >= c.dims[j]) reachable = false;
            if (v[j]) zero = false;
        }
        if (!reachable) continue;  // mesh: the source lies outside for every process
        Part p;
        p.phase = 0;
        p.round = i;
        p.slot = i;
        p.src_off = r.sdispl[i];
        p.dst_off = r.rdispl[i];
        p.len = r.len[i];
        std::memcpy(p.shift, v, sizeof(int) * g.d);
        for (int j = 0; j < g.d; ++j)
            if (!c.periodic[j]) p.check[j] = v[j];
        r.parts.push_back(p);
        if (zero) ++locals; else ++parts;
    }
    r.stats.rounds = g.s;
    r.stats.max_rounds_per_dim = g.s;
    r.stats.parts = parts;
    r.stats.local_copies = locals;
    r.inter_stride = 0;
    return ISO_SUCCESS;
}

// Assigns intermediate-buffer offsets to the slots flagged in `needs`; an offset keeps the
// misalignment (mod 16) of the slot's receive displacement so that copies between the two
// buffers can use wide accesses.
std::vector<int64_t> layout_inter(Request &r, const std::vector<char> &needs)
{
    std::vector<int64_t> off(needs.size(), -1);
    int64_t cur = 0;
    for (size_t i = 0; i < needs.size(); ++i) {
        if (!needs[i]) continue;
        int64_t mis = r.len[i] >= 16 ? (r.rdispl[i] & 15) : 0;
        int64_t a = r.len[i] >= 16 ? 16 : (r.len[i] >= 8 ? 8 : (r.len[i] >= 4 ? 4 : 1));
        cur = round_up(cur, a) + mis;
        off[i] = cur;
        cur += r.len[i];
    }
    r.inter_stride = round_up(cur, 16);
    return off;
}

int64_t offset_in(const Request &r, int buf, int slot, const std::vector<int64_t> &inter_off)
{
    if (buf == ISO_BUF_SEND) return r.sdispl[slot];
    if (buf == ISO_BUF_RECV) return r.rdispl[slot];
    return inter_off[slot];
}

// One hop of slot i under the alternating rule of Algorithm 1.
void emit_hop(Request &r, int phase, int round, int slot, const int *shift, int d,
              std::vector<int> &remaining, std::vector<int> &cur_buf,
              const std::vector<int64_t> &inter_off, std::vector<Part> &out)
{
    Part p;
    p.phase = phase;
    p.round = round;
    p.slot = slot;
    p.src_buf = cur_buf[slot];
    p.dst_buf = (remaining[slot] & 1) ? ISO_BUF_RECV : ISO_BUF_INTER;
    p.src_off = offset_in(r, p.src_buf, slot, inter_off);
    p.dst_off = offset_in(r, p.dst_buf, slot, inter_off);
    p.len = r.len[slot];
    std::memcpy(p.shift, shift, sizeof(int) * d);
    out.push_back(p);
    remaining[slot] -= 1;
    cur_buf[slot] = p.dst_buf;
}

// Packed intermediate storage.  Algorithm 1 lets a block alternate between the receive
// buffer and one intermediate buffer, each block staying at "its" slot; on a GPU that leaves
// every phase reading and writing isolated blocks scattered over three buffers.  Here every
// non-final hop of a block gets a place of its own in the intermediate buffer, and places are
// ordered by (phase that writes, phase that reads, slot): a phase then writes one contiguous
// region per process and reads a few contiguous regions, and the receive buffer is written
// only by final hops.  The hops, their order and the bytes moved are unchanged; the
// intermediate buffer grows from one place per multi-hop block to (hops - 1) places.
void pack_intermediates(Request &r, int s, bool final_by_dst)
{
    std::vector<std::vector<size_t>> chain(s);  // indices of a slot's hops, in execution order
    for (size_t k = 0; k < r.parts.size(); ++k) chain[r.parts[k].slot].push_back(k);
    struct Place { int write_phase, read_phase, read_round, slot, hop; };
    std::vector<Place> places;
    // Blocks that one round reads lie side by side: a process then fetches one contiguous
    // run per source process instead of pieces interleaved with those of other rounds.
    // Only where every block fills whole 32-byte sectors: with smaller blocks it is the
    // writers' pieces that get split, which measured slower.
    int64_t min_len = INT64_MAX;
    for (int i = 0; i < s; ++i)
        if (r.len[i] > 0) min_len = std::min(min_len, r.len[i]);
    bool by_round = min_len >= 32;
    if (r.knobs.pack_by_round >= 0) by_round = r.knobs.pack_by_round != 0;
    for (int i = 0; i < s; ++i)
        for (size_t j = 0; j + 1 < chain[i].size(); ++j)
            places.push_back(Place{r.parts[chain[i][j]].phase, r.parts[chain[i][j + 1]].phase,
                                   by_round ? r.parts[chain[i][j + 1]].round : 0, i, (int)j});
    std::sort(places.begin(), places.end(), [](const Place &a, const Place &b) {
        if (a.write_phase != b.write_phase) return a.write_phase < b.write_phase;
        if (a.read_phase != b.read_phase) return a.read_phase < b.read_phase;
        if (a.read_round != b.read_round) return a.read_round < b.read_round;
        return a.slot < b.slot;
    });
    int64_t cur = 0;
    for (const Place &pl : places) {
        const int64_t len = r.len[pl.slot];
        const bool co_aligned = ((r.sdispl[pl.slot] ^ r.rdispl[pl.slot]) & 15) == 0;
        const int64_t mis = (len >= 16 && co_aligned) ? (r.rdispl[pl.slot] & 15) : 0;
        const int64_t a = len >= 16 ? 16 : (len >= 8 ? 8 : (len >= 4 ? 4 : 1));
        cur = round_up(cur, a) + mis;
        Part &w = r.parts[chain[pl.slot][pl.hop]], &rd = r.parts[chain[pl.slot][pl.hop + 1]];
        w.dst_buf = ISO_BUF_INTER;
        w.dst_off = cur;
        rd.src_buf = ISO_BUF_INTER;
        rd.src_off = cur;
        cur += len;
    }
    for (int i = 0; i < s; ++i) {
        if (chain[i].empty()) continue;
        Part &first = r.parts[chain[i].front()], &last = r.parts[chain[i].back()];
        first.src_buf = ISO_BUF_SEND;
        first.src_off = r.sdispl[i];
        last.dst_buf = ISO_BUF_RECV;
        last.dst_off = r.rdispl[i];
    }
    r.inter_stride = round_up(cur, 16);
    // inside a phase, take the parts in the order of their source addresses
    // (the phase of the postponed final hops of 16-byte blocks in the order of the receive
    // buffer instead: whole-row stores and scattered loads measured 5 % faster there than
    // the other way round, 185 against 196 microseconds on the 8^5 torus)
    int last_phase = 0;
    for (const Part &p : r.parts) last_phase = std::max(last_phase, p.phase);
    std::stable_sort(r.parts.begin(), r.parts.end(), [&](const Part &a, const Part &b) {
        if (a.phase != b.phase) return a.phase < b.phase;
        if (final_by_dst && a.phase == last_phase) {
            if (a.dst_buf != b.dst_buf) return a.dst_buf < b.dst_buf;
            return a.dst_off < b.dst_off;
        }
        if (a.src_buf != b.src_buf) return a.src_buf < b.src_buf;
        return a.src_off < b.src_off;
    });
}

// Section V all-to-all: dimensions (or groups of consecutive dimensions) one after the
// other; inside a group one round per distinct non-zero projected coordinate vector.
int build_combining_alltoall(Request &r, const Geometry &g)
{
    const Comm &c = *r.comm;
    const Groups gr = make_groups(g.d, r.fusion);
    std::vector<int> hops(g.s, 0);
    std::vector<char> live(g.s, 1);  // false: empty block, or no process can ever receive it (mesh)
    bool mesh = false;
    for (int j = 0; j < g.d; ++j) mesh |= !c.periodic[j];
    for (int i = 0; i < g.s; ++i) {
        if (r.len[i] == 0) live[i] = 0;
        for (int j = 0; j < g.d; ++j)
            if (!c.periodic[j] && std::abs((int64_t)g.at(i)[j]) >= c.dims[j]) live[i] = 0;
        for (int k = 0; k < gr.n; ++k)
            if (group_nonzero(g.at(i), gr.begin[k], gr.begin[k + 1])) ++hops[i];
    }
    std::vector<char> needs(g.s, 0);
    for (int i = 0; i < g.s; ++i) needs[i] = live[i] && hops[i] >= 2;
    std::vector<int64_t> inter_off = layout_inter(r, needs);

    std::vector<int> remaining = hops, cur_buf(g.s, ISO_BUF_SEND);
    int round = 0, phase = 0, nmax = 0, parts = 0, locals = 0;
    std::vector<Part> locals_parts;
    for (int i = 0; i < g.s; ++i)
        if (live[i] && hops[i] == 0) { add_local_copy(r, i, locals_parts); ++locals; }

    for (int k = 0; k < gr.n; ++k) {
        const int j0 = gr.begin[k], j1 = gr.begin[k + 1];
        // bucket the neighbours by their coordinates in this group
        std::map<std::vector<int>, std::vector<int>, RoundOrder> buckets(RoundOrder{c.dims, c.periodic, j0, j1});
        for (int i = 0; i < g.s; ++i) {
            if (!live[i] || !group_nonzero(g.at(i), j0, j1)) continue;
            buckets[std::vector<int>(g.at(i) + j0, g.at(i) + j1)].push_back(i);
        }
        nmax = std::max<int>(nmax, (int)buckets.size());
        const size_t group_begin = r.parts.size();
        for (auto &b : buckets) {
            int shift[ISO_MAX_DIMS] = {0};
            for (int j = j0; j < j1; ++j) shift[j] = b.first[j - j0];
            for (int i : b.second) {
                emit_hop(r, phase, round, i, shift, g.d, remaining, cur_buf, inter_off, r.parts);
                ++parts;
            }
            ++round;
            if (r.fusion == 0) ++phase;
        }
        if (r.fusion != 0 && r.parts.size() > group_begin) {
            // rounds of one group touch disjoint slots: run them together, in slot order
            std::stable_sort(r.parts.begin() + group_begin, r.parts.end(),
                             [](const Part &a, const Part &b) { return a.slot < b.slot; });
            ++phase;
        }
    }
    if (mesh) {
        // Non-periodic dimensions: a block travels only if both its original sender and its
        // final receiver exist.  Seen from the process x that receives hop h of the block,
        // the sender is x minus the coordinates already applied and the receiver x plus the
        // ones still to come, so along a mesh dimension j the hop is performed iff
        // 0 <= x_j - check_j < p_j with check_j = +c_j (applied, this hop included) or -c_j.
        std::vector<std::vector<size_t>> chain(g.s);
        for (size_t k = 0; k < r.parts.size(); ++k) chain[r.parts[k].slot].push_back(k);
        for (int i = 0; i < g.s; ++i) {
            bool applied[ISO_MAX_DIMS] = {false};
            for (size_t k : chain[i]) {
                Part &p = r.parts[k];
                for (int j = 0; j < g.d; ++j)
                    if (p.shift[j]) applied[j] = true;
                for (int j = 0; j < g.d; ++j)
                    if (!c.periodic[j]) p.check[j] = applied[j] ? g.at(i)[j] : -g.at(i)[j];
            }
        }
    }
    // Blocks of at most 16 bytes: run every block's final hop in the last phase (a hop may
    // be postponed, only the order of a block's own hops matters), so that the receive
    // buffer is written by one launch, whole rows at a time, instead of in isolated
    // half-sector pieces by every phase.  Measured +40 % on the 8^5 torus with 16-byte
    // blocks; for blocks of 64 bytes and more the uneven phases cost 4-6 %, so they keep
    // the natural phases.
    bool lazy_final = r.layout == ISO_LAYOUT_PACKED && r.fusion != 0 && phase > 1;
    for (int i = 0; i < g.s; ++i)
        if (r.len[i] > 16) lazy_final = false;
    if (r.knobs.lazy_final >= 0)
        lazy_final = r.layout == ISO_LAYOUT_PACKED && r.fusion != 0 && phase > 1 && r.knobs.lazy_final != 0;
    if (lazy_final) {
        std::vector<int> last_hop(g.s, -1);
        for (size_t k = 0; k < r.parts.size(); ++k) last_hop[r.parts[k].slot] = (int)k;
        for (int i = 0; i < g.s; ++i)
            if (last_hop[i] >= 0) r.parts[last_hop[i]].phase = phase - 1;
        std::stable_sort(r.parts.begin(), r.parts.end(),
                         [](const Part &a, const Part &b) { return a.phase < b.phase; });
    }
    // on a mesh the receive buffer must not serve as scratch (an undelivered slot keeps its
    // contents), so the packed layout is used whatever was asked for
    bool full_units = true;  // every block fills whole 16-byte units
    for (int i = 0; i < g.s; ++i)
        if (r.len[i] > 0 && r.len[i] % 16 != 0) full_units = false;
    if (r.layout == ISO_LAYOUT_PACKED || mesh) pack_intermediates(r, g.s, lazy_final && full_units);
    // blocks for the process itself: one local copy, together with the first phase
    for (Part &p : locals_parts) p.phase = 0;
    r.parts.insert(r.parts.begin(), locals_parts.begin(), locals_parts.end());
    r.stats.rounds = round;
    r.stats.max_rounds_per_dim = nmax;
    r.stats.parts = parts;
    r.stats.local_copies = locals;
    return ISO_SUCCESS;
}

// Algorithm 1: hop-by-hop all-to-all between immediate torus neighbours.  Step h of the
// positive half of dimension j forwards every block with c^i_j > h by one hop; the negative
// half mirrors it.  A block is read from the send buffer only on its very first hop.
int build_torus_alltoall(Request &r, const Geometry &g)
{
    const Comm &c = *r.comm;
    std::vector<int> sym((size_t)g.s * g.d), hops(g.s, 0);
    for (int i = 0; i < g.s; ++i)
        for (int j = 0; j < g.d; ++j) {
            sym[(size_t)i * g.d + j] = symmetric_rep(g.at(i)[j], c.dims[j]);
            hops[i] += std::abs(sym[(size_t)i * g.d + j]);
        }
    std::vector<char> needs(g.s, 0);
    for (int i = 0; i < g.s; ++i) needs[i] = r.len[i] > 0 && hops[i] >= 2;
    std::vector<int64_t> inter_off = layout_inter(r, needs);
    std::vector<int> remaining = hops, cur_buf(g.s, ISO_BUF_SEND);
    int round = 0, nmax = 0, parts = 0, locals = 0;
    std::vector<Part> locals_parts;
    for (int i = 0; i < g.s; ++i)
        if (r.len[i] > 0 && hops[i] == 0) { add_local_copy(r, i, locals_parts); ++locals; }
    for (int j = 0; j < g.d; ++j) {
        int per_dim = 0;
        for (int sign = +1; sign >= -1; sign -= 2) {
            int reach = 0;
            for (int i = 0; i < g.s; ++i)
                if (r.len[i] > 0) reach = std::max(reach, sign * sym[(size_t)i * g.d + j]);
            for (int h = 0; h < reach; ++h) {
                int shift[ISO_MAX_DIMS] = {0};
                shift[j] = reduce_mod(sign, c.dims[j]);
                for (int i = 0; i < g.s; ++i) {
                    if (r.len[i] == 0 || sign * sym[(size_t)i * g.d + j] <= h) continue;
                    emit_hop(r, round, round, i, shift, g.d, remaining, cur_buf, inter_off, r.parts);
                    ++parts;
                }
                ++round;
                ++per_dim;
            }
        }
        nmax = std::max(nmax, per_dim);
    }
    for (Part &p : locals_parts) p.phase = 0;
    r.parts.insert(r.parts.begin(), locals_parts.begin(), locals_parts.end());
    r.stats.rounds = round;
    r.stats.max_rounds_per_dim = nmax;
    r.stats.parts = parts;
    r.stats.local_copies = locals;
    return ISO_SUCCESS;
}

// Section III-B / V allgather.  A trie node is a distinct prefix of the (reduced) offset
// vectors; a node whose last coordinate group is non-zero is produced in the round of that
// coordinate by reading its parent's storage one shift away; a zero edge forwards nothing
// and shares the parent's storage.  A node is stored in the receive slot of the first
// neighbour whose vector is the prefix padded with zeros, else in the intermediate buffer.
int build_combining_allgather(Request &r, const Geometry &g)
{
    const Comm &c = *r.comm;
    const Groups gr = make_groups(g.d, r.fusion);
    const int64_t m = g.s ? r.len[0] : 0;
    struct Store { int buf; int64_t off; };
    // Visiting order of the dimensions (Section III-B leaves it open; the result does not depend
    // on it).  order[k] is the dimension visited k-th; below, coordinate vectors, sizes and
    // periodicity are all taken in visiting order, and only shifts and check values are written
    // back by dimension.
    int order[ISO_MAX_DIMS], pdims[ISO_MAX_DIMS], pper[ISO_MAX_DIMS];
    for (int k = 0; k < g.d; ++k) {
        order[k] = r.dim_order[k];
        pdims[k] = c.dims[order[k]];
        pper[k] = c.periodic[order[k]];
    }
    std::vector<int> visited((size_t)g.s * g.d);
    for (int i = 0; i < g.s; ++i)
        for (int k = 0; k < g.d; ++k) visited[(size_t)i * g.d + k] = g.at(i)[order[k]];
    auto at = [&](int i) { return visited.data() + (size_t)i * g.d; };
    // Non-periodic dimensions (Section VII): the node of prefix Q exists at process x only if
    // the process x - (Q, 0, ..., 0) does, so a part that produces it carries, for every mesh
    // dimension already visited, the prefix's coordinate as its check value.  A node kept in
    // a receive slot is then written exactly where that slot's block is deliverable, and
    // elsewhere the slot keeps its contents.  A neighbour whose coordinate reaches across
    // the whole mesh can never be served and takes no part.
    bool mesh = false;
    for (int j = 0; j < g.d; ++j) mesh |= !pper[j];
    std::vector<char> dead(g.s, 0);
    for (int i = 0; i < g.s; ++i)
        for (int j = 0; j < g.d; ++j)
            if (!pper[j] && std::abs((int64_t)at(i)[j]) >= pdims[j]) dead[i] = 1;
    std::map<std::vector<int>, int> first_with_vector;  // full vector -> smallest slot
    for (int i = g.s - 1; i >= 0; --i)
        if (!dead[i]) first_with_vector[std::vector<int>(at(i), at(i) + g.d)] = i;

    std::map<std::vector<int>, Store> storage;  // prefix -> where that block lives
    storage[std::vector<int>()] = Store{ISO_BUF_SEND, 0};
    int64_t inter_cur = 0;
    int round = 0, phase = 0, nmax = 0, parts = 0, locals = 0;
    std::vector<Part> locals_parts;
    std::vector<char> served(g.s, 0);

    if (m > 0)
        for (int i = 0; i < g.s; ++i)
            if (!dead[i] && !group_nonzero(at(i), 0, g.d)) { add_local_copy(r, i, locals_parts); served[i] = 1; ++locals; }

    for (int k = 0; k < gr.n && m > 0; ++k) {
        const int j0 = gr.begin[k], j1 = gr.begin[k + 1];
        // rounds of this group: distinct non-zero coordinate keys
        std::map<std::vector<int>, int, RoundOrder> round_of(RoundOrder{pdims, pper, j0, j1});
        for (int i = 0; i < g.s; ++i)
            if (!dead[i] && group_nonzero(at(i), j0, j1)) round_of[std::vector<int>(at(i) + j0, at(i) + j1)] = 0;
        nmax = std::max<int>(nmax, (int)round_of.size());
        for (auto &kv : round_of) kv.second = round++;
        const size_t group_begin = r.parts.size();
        for (int i = 0; i < g.s; ++i) {
            if (dead[i]) continue;
            std::vector<int> prefix(at(i), at(i) + j1), parent(at(i), at(i) + j0);
            const Store src = storage.at(parent);
            if (!group_nonzero(at(i), j0, j1)) {
                storage.emplace(prefix, src);  // zero edge: nothing moves
                continue;
            }
            int shift[ISO_MAX_DIMS] = {0};
            for (int j = j0; j < j1; ++j) shift[order[j]] = at(i)[j];
            const int rnd = round_of.at(std::vector<int>(at(i) + j0, at(i) + j1));
            auto emit = [&](int slot, Store dst) {
                Part p;
                p.phase = r.fusion == 0 ? rnd : phase;
                p.round = rnd;
                p.slot = slot;
                p.src_buf = src.buf;
                p.src_off = src.off;
                p.dst_buf = dst.buf;
                p.dst_off = dst.off;
                p.len = m;
                std::memcpy(p.shift, shift, sizeof(shift));
                if (mesh)
                    for (int j = 0; j < j1; ++j)
                        if (!pper[j]) p.check[order[j]] = at(i)[j];
                r.parts.push_back(p);
                ++parts;
            };
            if (!storage.count(prefix)) {
                // new trie node: choose its storage and produce it
                std::vector<int> padded(prefix);
                padded.resize(g.d, 0);
                auto it = first_with_vector.find(padded);
                Store dst;
                int slot = -1;
                if (it != first_with_vector.end()) {
                    slot = it->second;
                    dst = Store{ISO_BUF_RECV, r.rdispl[slot]};
                    served[slot] = 1;
                } else {
                    dst = Store{ISO_BUF_INTER, inter_cur};
                    inter_cur += round_up(m, 16);
                }
                storage.emplace(prefix, dst);
                emit(slot, dst);
            }
            // a neighbour whose vector ends here but whose slot does not hold the node
            // (a repeated vector) receives its own copy in the same round
            if (!served[i] && !group_nonzero(at(i), j1, g.d)) {
                emit(i, Store{ISO_BUF_RECV, r.rdispl[i]});
                served[i] = 1;
            }
        }
        if (r.fusion != 0 && r.parts.size() > group_begin) ++phase;
    }
    if (r.fusion == 0) {
        // per-round launches: parts were emitted in slot order, bring them into round order
        std::stable_sort(r.parts.begin(), r.parts.end(),
                         [](const Part &a, const Part &b) { return a.phase < b.phase; });
    }
    for (Part &p : locals_parts) p.phase = 0;
    r.parts.insert(r.parts.begin(), locals_parts.begin(), locals_parts.end());
    r.inter_stride = inter_cur;
    r.stats.rounds = round;
    r.stats.max_rounds_per_dim = nmax;
    r.stats.parts = parts;
    r.stats.local_copies = locals;
    return ISO_SUCCESS;
}

void compress_phases(std::vector<Part> &parts, int &phases)
{
    int next = -1, last = -1;
    for (Part &p : parts) {
        if (p.phase != last) { last = p.phase; ++next; }
        p.phase = next;
    }
    phases = next + 1;
}

}  // namespace

// The allgather's trie may visit the dimensions in any order (Section III-B).  The last
// dimension visited produces the most blocks: two thirds of them for a Moore neighbourhood of
// radius 1.  Visiting dimension 0 LAST makes that phase copy runs of consecutive receive slots
// (the neighbours are listed with the last coordinate fastest, so the children of consecutive
// parents are consecutive slots), where visiting it first leaves every parent between its
// own children and each 64-byte load drags in the line around it.  The price: the last phase
// then reads from processes a whole plane of dimension 0 away, so a parent that many children
// read (one per distinct non-zero coordinate) comes from device memory every time instead of
// from the cache.  Measured (64-byte blocks, last-to-first against first-to-last): 2 distinct
// coordinates 97 against 143 microseconds (16^4 torus) and 19.1 against 20.6 (32^3), 3 (positive
// octant, r=3) 32 against 40, 6 (Moore r=3) 190 against 206, 14 (Chebyshev shells 3 and 7)
// 1004 against 800.  Hence: last-to-first up to 8 distinct coordinates in dimension 0.
void default_dimension_order(Request &r)
{
    const Comm &c = *r.comm;
    for (int k = 0; k < ISO_MAX_DIMS; ++k) r.dim_order[k] = k;
    if (r.kind != ISO_KIND_ALLGATHER || c.d < 2) return;
    bool reversed;
    if (r.knobs.ag_order >= 0) {
        reversed = r.knobs.ag_order == 1;
    } else {
        std::vector<int> values;
        for (int i = 0; i < c.s; ++i) {
            const int v = c.coords[(size_t)i * c.d];
            const int x = c.periodic[0] ? reduce_mod(v, c.dims[0]) : v;
            if (x != 0 && std::find(values.begin(), values.end(), x) == values.end()) values.push_back(x);
        }
        reversed = values.size() <= 8;
    }
    if (reversed)
        for (int k = 0; k < c.d; ++k) r.dim_order[k] = c.d - 1 - k;
}

int build_schedule(Request &r)
{
    const Comm &c = *r.comm;
    Geometry g;
    g.d = c.d;
    g.s = c.s;
    g.red.resize((size_t)c.s * c.d);
    bool mesh = false;
    for (int j = 0; j < c.d; ++j) mesh |= !c.periodic[j];
    for (int i = 0; i < c.s; ++i)
        for (int j = 0; j < c.d; ++j) {
            int v = c.coords[(size_t)i * c.d + j];
            g.red[(size_t)i * c.d + j] = c.periodic[j] ? reduce_mod(v, c.dims[j]) : v;
        }
    // meshes: the direct and the combining schedules; Algorithm 1 as printed alternates a
    // block between its receive slot and the intermediate buffer, which an undelivered
    // slot that must keep its contents does not allow
    if (mesh && r.alg == ISO_ALG_TORUS) return ISO_ERR_ARG;
    const bool gather = r.kind == ISO_KIND_ALLGATHER;
    if (r.alg == ISO_ALG_TORUS && gather) return ISO_ERR_ARG;
    if (r.alg != ISO_ALG_COMBINING && r.alg != ISO_ALG_DIRECT && r.alg != ISO_ALG_TORUS) return ISO_ERR_ARG;
    if (r.fusion < 0) return ISO_ERR_ARG;

    r.parts.clear();
    r.inter_stride = 0;
    Iso_stats st{};
    r.stats = st;
    int rc;
    if (r.alg == ISO_ALG_DIRECT) rc = build_direct(r, g);
    else if (r.alg == ISO_ALG_TORUS) rc = build_torus_alltoall(r, g);
    else if (gather) rc = build_combining_allgather(r, g);
    else rc = build_combining_alltoall(r, g);
    if (rc != ISO_SUCCESS) return rc;

    // phase numbers must be non-decreasing in execution order
    std::stable_sort(r.parts.begin(), r.parts.end(),
                     [](const Part &a, const Part &b) { return a.phase < b.phase; });
    int phases = 0;
    compress_phases(r.parts, phases);

    int64_t payload = 0, moved = 0;
    for (int i = 0; i < c.s; ++i) payload += r.len[i];
    for (const Part &p : r.parts) moved += p.len;
    r.stats.kind = r.kind;
    r.stats.algorithm = r.alg;
    r.stats.fusion_level = r.fusion;
    r.stats.d = c.d;
    r.stats.s = c.s;
    r.stats.phases = phases;
    r.stats.P = c.P;
    r.stats.send_stride = r.send_stride;
    r.stats.recv_stride = r.recv_stride;
    r.stats.inter_stride = r.inter_stride;
    r.stats.bytes_min = 2 * c.P * payload;
    r.stats.bytes_moved = 2 * c.P * moved;
    return validate_schedule(r);
}

int validate_schedule(const Request &r)
{
    struct Range { int64_t lo, hi; bool write; };
    const int64_t stride[3] = {r.send_stride, r.recv_stride, r.inter_stride};
    size_t begin = 0;
    while (begin < r.parts.size()) {
        size_t end = begin;
        while (end < r.parts.size() && r.parts[end].phase == r.parts[begin].phase) ++end;
        std::vector<Range> ranges[3];
        for (size_t k = begin; k < end; ++k) {
            const Part &p = r.parts[k];
            if (p.len <= 0 || p.src_off < 0 || p.dst_off < 0) return ISO_ERR_STATE;
            if (p.src_buf < 0 || p.src_buf > 2 || p.dst_buf < 1 || p.dst_buf > 2) return ISO_ERR_STATE;
            if (p.src_off + p.len > stride[p.src_buf] || p.dst_off + p.len > stride[p.dst_buf]) return ISO_ERR_STATE;
            ranges[p.src_buf].push_back(Range{p.src_off, p.src_off + p.len, false});
            ranges[p.dst_buf].push_back(Range{p.dst_off, p.dst_off + p.len, true});
        }
        for (auto &v : ranges) {
            std::sort(v.begin(), v.end(), [](const Range &a, const Range &b) { return a.lo < b.lo; });
            // a write may not overlap anything else; reads may overlap reads
            int64_t write_hi = -1, any_hi = -1;
            for (const Range &x : v) {
                if (x.lo < write_hi) return ISO_ERR_OVERLAP;
                if (x.write && x.lo < any_hi) return ISO_ERR_OVERLAP;
                any_hi = std::max(any_hi, x.hi);
                if (x.write) write_hi = std::max(write_hi, x.hi);
            }
        }
        begin = end;
    }
    return ISO_SUCCESS;
}

// --------------------------------------------------------------------------------------
// Lowering to kernel launches.
namespace {

int pow2_alignment(int64_t x)
{
    if (x == 0) return 16;
    int a = 1;
    while (a < 16 && (x & a) == 0) a <<= 1;
    return a;
}

int common_alignment(std::initializer_list<int64_t> xs)
{
    int a = 16;
    for (int64_t x : xs) a = std::min(a, pow2_alignment(x));
    return a;
}

}  // namespace

// Whether the schedule can run slab by slab (see plan_slabs in iso_api.cu): every part that
// shifts along dimension 0 reads the send buffer, all dimensions periodic, at least four planes.
static bool slabs_possible(const Request &r)
{
    const Comm &c = *r.comm;
    if (c.d < 2 || c.dims[0] < 4) return false;
    for (int j = 0; j < c.d; ++j)
        if (!c.periodic[j]) return false;
    for (const Part &p : r.parts)
        if (p.shift[0] != 0 && p.src_buf != ISO_BUF_SEND) return false;
    return true;
}

int lower_schedule(Request &r, uintptr_t send_addr, uintptr_t recv_addr, uintptr_t inter_addr)
{
    const Comm &c = *r.comm;
    // From which part length on the bulk-copy kernel is used.  Asked for, or: 512 bytes (the
    // measured crossover of one launch against one launch) - except where the library may run
    // the schedule in slabs of its own choice (an all-to-all with intermediate blocks) and can
    // make the slabs small enough for the L2 (choose_slab_plan: 52 MB written per launch, at
    // most 128 slabs of at least two planes and 512 processes): there the vector kernel moves
    // everything, because only it runs well in launches of a slab's size, and a slab's
    // intermediate blocks are then read back out of the L2.  Measured on the 256x256 torus,
    // Moore r=2, bulk kernel in one launch per phase against vector kernel in slabs: 512-byte
    // blocks 438 against 391 microseconds, 1 KB 820 against 783, 2 KB 1668 against 1566, 4 KB
    // 3295 against 3157 (128 slabs).
    if (r.bulk_threshold_asked >= 0) {
        r.bulk_threshold = r.bulk_threshold_asked;
    } else {
        bool own_slabs = r.kind != ISO_KIND_ALLGATHER && r.inter_stride > 0 && r.slab_request == 0 && r.knobs.slabs < 0 &&
                         !r.persistent && r.wave_request == 0 && slabs_possible(r);
        if (own_slabs) {
            const double written = (double)r.stats.bytes_moved / 2.0 / (double)std::max(1, r.stats.phases);
            int64_t need = 1;
            while (need < kMaxOwnSlabs && written / (double)need > kSlabLaunchBytes) need *= 2;
            own_slabs = written / (double)need <= kSlabLaunchBytes && need * 2 <= c.dims[0] && c.P / need >= 512;
        }
        r.bulk_threshold = own_slabs ? 0 : 512;
    }
    const int64_t stride[3] = {r.send_stride, r.recv_stride, r.inter_stride};
    const int64_t addr[3] = {(int64_t)send_addr, (int64_t)recv_addr, (int64_t)inter_addr};
    r.launches.clear();
    int64_t bulk_bytes = 0;
    int64_t fan_saved = 0;  // bytes per process that sender-side launches do not read again

    size_t begin = 0;
    while (begin < r.parts.size()) {
        size_t end = begin;
        while (end < r.parts.size() && r.parts[end].phase == r.parts[begin].phase) ++end;

        // Allgather phase in its sender-side form: every part moves along one and the same
        // periodic dimension (or not at all), in whole 16-byte units below the bulk threshold,
        // and the request runs neither in slabs nor in a one-launch mode (a launch then reads
        // the rows it is given and writes into other rows).
        // Measured (64-byte blocks): +7-8 % where a block has two or three copies and the phase is
        // large (80 neighbours on 16^4, the positive octant), -8 % on the small 32^3 torus and
        // -13 to -26 % where a block has six or more copies (radius 3, the shells), because a
        // gather writes whole rows in one pass while this form scatters 64-byte pieces over
        // several rows.  Hence, when left to the library (sender_side 1): only phases in which
        // no block has more than kFanDsts copies and that write at least 64 MiB.
        if (r.kind == ISO_KIND_ALLGATHER && r.sender_side > 0 && r.wave_request == 0 && !r.persistent &&
            r.slab_request < 2 && r.knobs.slabs < 2 && r.chains_request < 2 && r.knobs.chains < 2) {
            int dim = -1;
            bool ok = true;
            for (size_t k = begin; k < end && ok; ++k) {
                const Part &p = r.parts[k];
                const int base = common_alignment({stride[p.src_buf], stride[p.dst_buf], addr[p.src_buf], addr[p.dst_buf],
                                                   p.src_off, p.dst_off, p.len});
                if (base != 16 || (r.bulk_threshold > 0 && p.len >= r.bulk_threshold)) ok = false;
                for (int j = 0; j < c.d; ++j) {
                    if (p.check[j]) ok = false;
                    if (!p.shift[j]) continue;
                    if (!c.periodic[j] || (dim >= 0 && dim != j)) ok = false;
                    dim = j;
                }
            }
            // at least one parent must feed two destinations, else the gather form is as good
            std::map<std::pair<int, int64_t>, size_t> parent_of;
            LaunchPlan L;
            if (ok) {
                for (size_t k = begin; k < end; ++k) {
                    const Part &p = r.parts[k];
                    auto key = std::make_pair(p.src_buf, p.src_off);
                    auto it = parent_of.find(key);
                    size_t at;
                    if (it == parent_of.end() || (int)L.fans[it->second].dsts.size() >= kFanDsts) {
                        FanParent f;
                        f.src_buf = p.src_buf;
                        f.src_off = p.src_off;
                        f.len = p.len;
                        at = L.fans.size();
                        L.fans.push_back(f);
                        parent_of[key] = at;
                    } else {
                        at = it->second;
                    }
                    if (L.fans[at].len != p.len) { ok = false; break; }
                    L.fans[at].dsts.push_back(FanDst{p.dst_buf, p.dst_off, dim >= 0 ? p.shift[dim] : 0});
                }
            }
            if (ok && r.sender_side == 1) {
                int64_t written = 0;
                for (size_t k = begin; k < end; ++k) written += r.parts[k].len;
                if (c.P * written < (64ll << 20) || parent_of.size() != L.fans.size()) ok = false;
            }
            if (ok && L.fans.size() < end - begin) {
                // destinations of a descriptor in the order of their shift, so that the e-th
                // stores of a warp go to the same process
                uint64_t units = 0;
                for (FanParent &f : L.fans) {
                    std::stable_sort(f.dsts.begin(), f.dsts.end(), [](const FanDst &a, const FanDst &b) { return a.c < b.c; });
                    units += (uint64_t)(f.len / 16);
                }
                if (units <= 0x7fffffffull) {
                    L.kernel = KERNEL_FAN;
                    L.width = 16;
                    L.phase = r.parts[begin].phase;
                    uint32_t first = 0;
                    for (size_t k = begin; k < end; ++k) {  // the same copies as parts, for Iso_request_get_parts
                        LoweredPart lp;
                        lp.p = r.parts[k];
                        lp.width = 16;
                        lp.first_unit = first;
                        lp.units = (uint32_t)(lp.p.len / 16);
                        first += lp.units;
                        L.parts.push_back(lp);
                    }
                    L.units_per_proc = (uint32_t)units;
                    if (dim >= 0) { L.used_dim[0] = dim; L.n_used = 1; }
                    L.max_nnz = L.n_used;
                    L.chunk_units = (uint32_t)std::min<uint64_t>(units, 1024);
                    L.rows_per_pass = std::max<uint32_t>(1, 1024 / L.chunk_units);
                    L.threads = (int)((L.chunk_units * L.rows_per_pass + 31) / 32 * 32);
                    L.grid = std::max<int64_t>(1, std::min<int64_t>((c.P + L.rows_per_pass - 1) / L.rows_per_pass, (int64_t)r.sm_count));
                    L.tile_procs = 1;
                    L.smem = (size_t)kWideDepth * L.threads * 16;
                    // bytes this launch moves: every parent read once per descriptor, every destination written
                    for (const FanParent &f : L.fans) fan_saved += (int64_t)(f.dsts.size() - 1) * f.len;
                    r.launches.push_back(std::move(L));
                    begin = end;
                    continue;
                }
            }
        }

        // whether this phase may run as one launch of mixed unit widths
        bool allow_mixed = r.wave_request == 0 && !r.persistent;
        if (r.knobs.mixed >= 0) allow_mixed = allow_mixed && r.knobs.mixed != 0;
        // split every part into pieces that share one alignment class
        // cls: width class of the launch (0: mixed widths); base: alignment of the rows it touches
        struct Piece { Part p; int kernel; int width; int cls; int base; };
        std::vector<Piece> pieces;
        for (size_t k = begin; k < end; ++k) {
            const Part &p = r.parts[k];
            const int base = common_alignment({stride[p.src_buf], stride[p.dst_buf], addr[p.src_buf], addr[p.dst_buf]});
            auto push = [&](int64_t rel, int64_t len) {
                if (len <= 0) return;
                Piece q;
                q.p = p;
                q.p.src_off = p.src_off + rel;
                q.p.dst_off = p.dst_off + rel;
                q.p.len = len;
                q.width = std::min(base, common_alignment({q.p.src_off, q.p.dst_off, len}));
                q.kernel = (q.width == 16 && r.bulk_threshold > 0 && len >= r.bulk_threshold) ? KERNEL_BULK : KERNEL_VEC;
                q.cls = q.width;
                q.base = base;
                pieces.push_back(q);
            };
            const bool co_aligned = base == 16 && ((p.src_off - p.dst_off) & 15) == 0;
            // ragged ends are cut into pieces of at most 4 bytes: with 8-byte end pieces the
            // irregular 64x64x32 workload measured 8 % slower (1.70 against 1.57 ms)
            const int64_t split_cap = 4;
            if (co_aligned && allow_mixed && ((p.src_off & 15) || (p.len & 15))) {
                // the launch of mixed widths takes any unit width: cut the ragged ends into
                // few aligned power-of-two pieces (a 15-byte head at offset 1 is
                // 1 + 2 + 4 + 4 + 4) around a body of whole 16-byte units
                int64_t rel = 0;
                while (rel < p.len && ((p.src_off + rel) & 15)) {
                    int64_t a = (p.src_off + rel) & -(p.src_off + rel);  // lowest set bit
                    a = std::min(a, split_cap);
                    while (a > p.len - rel) a >>= 1;
                    push(rel, a);
                    rel += a;
                }
                const int64_t body = (p.len - rel) / 16 * 16;
                push(rel, body);
                rel += body;
                for (int64_t a = split_cap; a >= 1; a >>= 1)
                    while (p.len - rel >= a) {
                        push(rel, a);
                        rel += a;
                    }
            } else if (co_aligned && p.len >= 48 && ((p.src_off & 15) || (p.len & 15))) {
                int64_t head = (16 - (p.src_off & 15)) & 15;
                int64_t body = (p.len - head) / 16 * 16;
                push(0, head);
                push(head, body);
                push(head + body, p.len - head - body);
            } else {
                push(0, p.len);
            }
        }

        // a vector class that carries next to nothing per process is not worth a launch of
        // its own: its pieces join the next narrower class that is in use
        // (only where every width takes a launch of its own: in a launch of mixed widths a
        // piece keeps its widest unit)
        for (int width = 16; width > 1 && !allow_mixed; width >>= 1) {
            int64_t bytes = 0;
            for (const Piece &q : pieces)
                if (q.kernel == KERNEL_VEC && q.width == width) bytes += q.p.len;
            if (bytes == 0 || bytes >= 128) continue;
            int narrower = 0;
            for (int w2 = width >> 1; w2 >= 1 && !narrower; w2 >>= 1)
                for (const Piece &q : pieces)
                    if (q.kernel == KERNEL_VEC && q.width == w2) { narrower = w2; break; }
            if (!narrower) continue;
            for (Piece &q : pieces)
                if (q.kernel == KERNEL_VEC && q.width == width) q.width = q.cls = narrower;
        }

        // Ragged rows (pieces of several widths in one phase): one launch of mixed unit
        // widths for all of them instead of one launch per width, so that pieces which share
        // a 32-byte sector are moved together.  Parts below 4 KB that would have gone to the
        // bulk kernel join it; they lie between the small pieces.  1- and 2-byte pieces take
        // part where every row starts on a 4-byte boundary (they fetch their aligned word).
        {
            auto eligible = [](const Piece &q) { return q.kernel == KERNEL_VEC && (q.width >= 4 || q.base >= 4); };
            int classes = 0;
            for (int width = 16; width >= 1; width >>= 1)
                for (const Piece &q : pieces)
                    if (eligible(q) && q.width == width) { ++classes; break; }
            if (classes >= 2 && allow_mixed)
                for (Piece &q : pieces) {
                    if (q.kernel == KERNEL_BULK && q.p.len < 4096) q.kernel = KERNEL_VEC;
                    if (eligible(q)) q.cls = 0;
                }
        }

        // parts of one launch with their unit ranges, the dimensions the launch shifts along
        // and the coarse unit -> part lookup
        auto fill_parts = [&](LaunchPlan &L, const std::vector<Piece> &src, size_t lo, size_t hi, int kernel, int64_t unit) -> int {
            uint64_t units = 0;
            bool uniform = true;
            bool used[ISO_MAX_DIMS] = {false};
            for (size_t k = lo; k < hi; ++k) {
                LoweredPart lp;
                lp.p = src[k].p;
                lp.width = kernel == KERNEL_BULK ? (int)unit : src[k].width;
                uint64_t n = (uint64_t)((lp.p.len + lp.width - 1) / lp.width);
                if (units + n > 0x7fffffffull) return ISO_ERR_COUNT;
                lp.first_unit = (uint32_t)units;
                lp.units = (uint32_t)n;
                units += n;
                if (!L.parts.empty() && L.parts[0].units != lp.units) uniform = false;
                int nnz = 0;
                for (int j = 0; j < c.d; ++j)
                    if (lp.p.shift[j] || lp.p.check[j]) { used[j] = true; ++nnz; }
                L.max_nnz = std::max(L.max_nnz, nnz);
                L.parts.push_back(lp);
            }
            L.units_per_proc = (uint32_t)units;
            L.uniform_units = uniform ? L.parts[0].units : 0;
            for (int j = 0; j < c.d; ++j)
                if (used[j]) L.used_dim[L.n_used++] = j;
            if (!uniform) {
                int shift = 0;
                while ((units >> shift) + 1 > 16384) ++shift;
                L.lookup_shift = shift;
                size_t n = (size_t)(units >> shift) + 1;
                L.lookup.resize(n);
                size_t t = 0;
                for (size_t e = 0; e < n; ++e) {
                    uint64_t u = (uint64_t)e << shift;
                    while (t + 1 < L.parts.size() && L.parts[t + 1].first_unit <= u) ++t;
                    L.lookup[e] = (uint16_t)t;
                }
            }
            return ISO_SUCCESS;
        };

        // one launch per (kernel, width) class, in a fixed order
        for (int kernel = 0; kernel < 2; ++kernel) {
            for (int width : {0, 16, 8, 4, 2, 1}) {  // 0: the launch of mixed unit widths
                std::vector<Piece> cls;
                std::vector<std::pair<size_t, size_t>> ranges;
                for (const Piece &q : pieces)
                    if (q.kernel == kernel && q.cls == width) cls.push_back(q);
                // Launch of mixed widths: the long 16-byte-aligned bodies among its pieces are
                // handed to one extra warp of the CTA that moves them with bulk copies, while
                // the other warps move the ragged rest (see iso_gather_rows_hybrid).
                std::vector<Piece> longs;
                if (kernel == KERNEL_VEC && width == 0 && r.hybrid && r.bulk_threshold_asked != 0 && c.d <= 3) {
                    bool plain = true;  // periodic dimensions only
                    for (const Piece &q : cls)
                        for (int j = 0; j < c.d; ++j) plain = plain && !q.p.check[j];
                    std::vector<Piece> rest;
                    for (const Piece &q : cls) (plain && q.width == 16 && q.p.len >= kHybridMinBytes ? longs : rest).push_back(q);
                    int64_t rest_units = 0;
                    for (const Piece &q : rest) rest_units += q.p.len / q.width;
                    if (!longs.empty() && !rest.empty() && rest_units <= kMaxVecUnits) cls.swap(rest);
                    else longs.clear();
                }
                // bulk side of such a launch: chunks of 1024 bytes if every long piece has as many,
                // else 512; two stages and two barriers per lane of one warp
                int64_t side_chunk = 1024;
                for (const Piece &q : longs) if (q.p.len < 1024) side_chunk = 512;
                // bulk warps: as many lanes as fill the staging area with two chunks each (measured with
                // ONE bulk warp, 32 KB in flight per SM: 2.8 times slower than without the split - a
                // bulk copy through shared memory occupies its stage for several microseconds)
                const size_t side_lanes = kHybridStageBytes / (2 * (size_t)side_chunk);
                const size_t side_smem = longs.empty() ? 0 : side_lanes * 2 * (size_t)side_chunk + side_lanes * 2 * 8;
                // a vector launch holds at most kMaxVecUnits unit positions per process (each
                // gets a descriptor): cut longer lists, splitting a piece at a unit boundary
                if (kernel == KERNEL_VEC) {
                    const int64_t cap = kMaxVecUnits;
                    std::vector<Piece> cut;
                    std::vector<size_t> bounds(1, 0);
                    int64_t used_units = 0;
                    for (Piece q : cls) {
                        while (q.p.len > 0) {
                            const int width = q.width;  // the piece's own unit width
                            int64_t n = q.p.len / width;
                            int64_t room = cap - used_units;
                            if (room == 0) { bounds.push_back(cut.size()); used_units = 0; room = cap; }
                            int64_t take = std::min(n, room);
                            Piece head = q;
                            head.p.len = take * width;
                            cut.push_back(head);
                            used_units += take;
                            q.p.src_off += take * width;
                            q.p.dst_off += take * width;
                            q.p.len -= take * width;
                        }
                    }
                    bounds.push_back(cut.size());
                    cls.swap(cut);
                    for (size_t b = 0; b + 1 < bounds.size(); ++b)
                        if (bounds[b] < bounds[b + 1]) ranges.push_back({bounds[b], bounds[b + 1]});
                } else {
                    const size_t max_parts = 60000;
                    for (size_t lo = 0; lo < cls.size(); lo += max_parts)
                        ranges.push_back({lo, std::min(cls.size(), lo + max_parts)});
                }
                for (const auto &range : ranges) {
                    const size_t lo = range.first, hi = range.second;
                    LaunchPlan L;
                    L.kernel = kernel;
                    L.phase = r.parts[begin].phase;
                    int64_t unit = width;  // 0 for mixed widths: every part then counts in its own
                    if (kernel == KERNEL_BULK) {
                        int64_t min_len = INT64_MAX;
                        for (size_t k = lo; k < hi; ++k) min_len = std::min(min_len, cls[k].p.len);
                        unit = 256;
                        while (unit * 2 <= min_len && unit < 2048) unit *= 2;
                        if (r.knobs.bulk_chunk) {
                            const int64_t v = r.knobs.bulk_chunk;
                            if (v >= 16 && v <= 16384 && v % 16 == 0) unit = v;
                        }
                    }
                    L.width = (int)unit;
                    {
                        int rc_fill = fill_parts(L, cls, lo, hi, kernel, unit);
                        if (rc_fill != ISO_SUCCESS) return rc_fill;
                    }
                    const uint64_t units = L.units_per_proc;
                    if (kernel == KERNEL_BULK)
                        for (const LoweredPart &lp : L.parts) bulk_bytes += lp.p.len;
                    // many shifted dimensions in the launch, few per part: the kernel then
                    // tests per row only the dimensions a unit moves along
                    {
                        bool torus = true;
                        for (int k = 0; k < L.n_used; ++k) torus = torus && c.periodic[L.used_dim[k]];
                        L.compact = kernel == KERNEL_VEC && (width >= 4 || width == 0) && L.n_used > 3 && L.max_nnz < L.n_used &&
                                    torus && !r.persistent;  // (the pipelined one-launch kernel does take compact launches)
                    }
                    // geometry
                    (void)width;
                    int64_t tp;
                    int64_t grid;
                    uint32_t whole_row_slots = 1;  // rows a CTA would hold if it covered whole rows
                    if (kernel == KERNEL_VEC) {
                        // a row slot covers up to 256 unit positions; short rows share a CTA
                        // 16-byte launches with long rows use CTAs of up to 1024 threads
                        // 16-byte and mixed launches run in CTAs of up to 1024 threads, one per SM
                        // (measured against four CTAs of 256 threads: 36.1 against 40.3 microseconds
                        // per all-to-all on the 32^3 torus, 161 against 184 on the 8^5 torus);
                        // ISO_VEC_THREADS=256 or 512 selects the narrower shapes
                        uint32_t max_threads = (width == 16 || width == 0) ? 1024 : 256;
                        if (!longs.empty())  // leave a warp and the staging area to the bulk side
                            max_threads = std::min<uint32_t>((uint32_t)(1024 - side_lanes),
                                                             (uint32_t)((227 * 1024 - side_smem - 16 * 1024) / (kHybridDepth * 16) / 32 * 32));
                        if (r.knobs.vec_threads && longs.empty()) {
                            const int v = r.knobs.vec_threads;
                            if ((v == 256 || v == 512) && max_threads == 1024) max_threads = units > 256 ? 1024 : (uint32_t)v;
                        }
                        L.chunk_units = (uint32_t)std::min<uint64_t>(units, max_threads);
                        L.rows_per_pass = std::max<uint32_t>(1, max_threads / L.chunk_units);
                        whole_row_slots = L.rows_per_pass;
                        // rows longer than a CTA: equal column chunks, the CTAs dealt to them (not in the
                        // one-launch modes, whose grids are sized elsewhere, nor with a bulk side)
                        // Measured on launches that shift along one dimension: shells 3.59 -> 3.21 ms, Moore d=3
                        // r=3 0.617 -> 0.544 ms, shells allgather 0.879 -> 0.797 ms; the one-pass direct launches
                        // (three wrap tests per row) lost 4 % and keep whole rows.  Splitting shorter rows to
                        // fill the CTA's thread slots (690 unit positions as 3 chunks x 4 rows), or into more
                        // chunks than needed, measured slower (irregular 64x64x32: 1.54 -> 1.60 ms; Moore r=3
                        // allgather 0.204 -> 0.235 ms).
                        L.col_split = 1;
                        if (max_threads == 1024 && units > max_threads && L.n_used <= 2 && longs.empty() && !r.persistent &&
                            r.wave_request == 0 && r.knobs.col_split) {
                            const uint32_t ncol = (uint32_t)((units + max_threads - 1) / max_threads);
                            L.col_split = (int)ncol;
                            L.chunk_units = (uint32_t)(((units + ncol - 1) / ncol + 31) / 32 * 32);
                            L.rows_per_pass = 1;
                        }
                        L.threads = (int)((L.chunk_units * L.rows_per_pass + 31) / 32 * 32);
                        // CTAs of fewer than 256 threads: as many per SM as keep 1024 threads resident
                        int per_sm = L.threads > 512 ? 1 : (L.threads > 256 ? 2 : std::min(16, std::max(4, 1024 / L.threads)));
                        if (!longs.empty()) per_sm = 1;
                        if (r.knobs.vec_ctas_per_sm) {
                            const int v = r.knobs.vec_ctas_per_sm;
                            if (v >= 1 && v <= 8 && L.threads <= 256) per_sm = v;
                        }
                        // persistent grid: CTA b takes the row groups b, b + grid, ...
                        grid = std::min<int64_t>((c.P + L.rows_per_pass - 1) / L.rows_per_pass,
                                                 (int64_t)r.sm_count * per_sm);
                        grid = std::max<int64_t>(grid, 1);
                        L.rows_hint = std::min<int64_t>((c.P + whole_row_slots - 1) / whole_row_slots, (int64_t)r.sm_count * per_sm) *
                                      whole_row_slots;
                        if (L.col_split > 1) {  // a multiple of the column chunks; the CTAs of one chunk share the rows
                            grid = std::max<int64_t>(1, std::min<int64_t>((c.P + L.rows_per_pass - 1) / L.rows_per_pass,
                                                                          r.sm_count / L.col_split)) * L.col_split;
                            L.rows_hint = std::max<int64_t>(1, r.sm_count / L.col_split);
                        }
                        tp = 1;
                    } else {
                        int threads = (int)(196608 / (2 * unit)) / 32 * 32;
                        L.threads = std::max(32, std::min(256, threads));
                        tp = std::max<int64_t>(1, (8 * (int64_t)L.threads + (int64_t)units - 1) / (int64_t)units);
                        tp = std::min<int64_t>(tp, 512);
                        tp = std::min<int64_t>(tp, std::max<int64_t>(1, c.P / ((int64_t)r.sm_count * 2)));
                        while (tp > 1 && (uint64_t)tp * units > 0x7fffffffull) tp /= 2;
                        if (r.knobs.bulk_tile) {
                            const int64_t v = r.knobs.bulk_tile;
                            if (v >= 1 && v <= 512 && (uint64_t)v * units <= 0x7fffffffull) tp = v;
                        }
                        grid = (c.P + tp - 1) / tp;
                    }
                    L.tile_procs = (int)tp;
                    L.grid = grid;
                    if (L.grid > 0x7fffffff) return ISO_ERR_DIMS;
                    L.smem = (size_t)L.n_used * (size_t)tp * sizeof(uint32_t);
                    if (kernel == KERNEL_VEC) {
                        const size_t depth = !longs.empty() ? kHybridDepth : (L.threads > 256 ? kWideDepth : kVecDepth);
                        L.smem = width >= 4 ? depth * L.threads * width : (width == 0 ? depth * L.threads * 16 : 0);
                    }
                    if (kernel == KERNEL_BULK)
                        L.smem = (L.smem + 15) / 16 * 16 + (size_t)L.threads * 2 * (size_t)unit + (size_t)L.threads * 2 * 8;
                    if (!longs.empty()) {
                        LaunchPlan S;
                        S.kernel = KERNEL_BULK;
                        S.phase = L.phase;
                        S.width = (int)side_chunk;
                        int rc_side = fill_parts(S, longs, 0, longs.size(), KERNEL_BULK, side_chunk);
                        if (rc_side != ISO_SUCCESS) return rc_side;
                        S.tile_procs = 1;
                        S.threads = (int)side_lanes;
                        S.smem = side_smem;
                        for (const LoweredPart &lp : S.parts) bulk_bytes += lp.p.len;
                        L.side.push_back(std::move(S));
                        longs.clear();
                    }
                    r.launches.push_back(std::move(L));
                }
            }
        }
        begin = end;
    }
    r.stats.launches = (int)r.launches.size();
    r.stats.bulk_bytes = 2 * c.P * bulk_bytes;
    int64_t moved = 0;
    for (const Part &p : r.parts) moved += p.len;
    r.stats.bytes_moved = c.P * (2 * moved - fan_saved);
    return ISO_SUCCESS;
}

}  // namespace iso
