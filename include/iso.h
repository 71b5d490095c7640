/*
 * iso.h - isomorphic, sparse neighbourhood collectives for P virtual processes on a
 * d-dimensional periodic torus, all resident in the memory of one CUDA device.
 *
 * The interface follows the persistent interface of the paper "Message-Combining
 * Algorithms for Isomorphic, Sparse Collective Communication" (Listings 1, 2 and 4):
 * a neighbourhood is created once from a list of relative coordinate vectors, an
 * `..._init` call binds buffers and precomputes a schedule, and `Iso_Start` runs it any
 * number of times.  MPI communicators and datatypes are replaced by plain integers.
 *
 * Model.  There are P = p_0 * ... * p_{d-1} processes; the process of rank r has the
 * coordinates of r written in the mixed radix (p_0, ..., p_{d-1}) with dimension d-1
 * varying fastest (the order of an MPI Cartesian communicator; the paper leaves it to
 * that communicator).  A buffer argument is a DEVICE pointer to the buffers of all P
 * processes, process-major: the buffer of process r starts `r * stride` bytes after the
 * pointer, where the stride is
 *     regular all-to-all : s * count * size            (s blocks back to back, Section II)
 *     allgather          : count * size   (send side), s * count * size (receive side)
 *     irregular          : max_i(displ_i + count_i * size), rounded up to a multiple of 16
 * `Iso_request_get_stats` reports the strides in use.
 *
 * Result (Section II).  With C^i the i-th relative coordinate vector and (-) the
 * component-wise subtraction modulo p_j, after `Iso_Start` + `Iso_wait`
 *     all-to-all : block i of process R's receive buffer = block i of the send buffer of R (-) C^i
 *     allgather  : block i of process R's receive buffer = the send block of R (-) C^i.
 *
 * Every function returns ISO_SUCCESS (0) or a positive ISO_ERR_* code; no exception or
 * abort crosses this boundary and output arguments are left untouched on failure.
 * Unless stated otherwise all pointer arguments other than buffers are HOST pointers that
 * are only read during the call.  The library is not thread safe per object: use one
 * request from one host thread at a time.
 */
#ifndef ISO_H
#define ISO_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ISO_MAX_DIMS 8

typedef struct Iso_comm_s *Iso_comm;       /* neighbourhood object, library owned */
typedef struct Iso_request_s *Iso_request; /* persistent collective, library owned */

/* Basic datatypes only carry a size: the payload is moved as opaque bytes.  Any positive
 * value is accepted and read as "bytes per element". */
typedef int Iso_datatype;
#define ISO_BYTE 1
#define ISO_INT32 4
#define ISO_FLOAT 4
#define ISO_DOUBLE 8

enum {
    ISO_SUCCESS = 0,
    ISO_ERR_ARG = 1,     /* null pointer, negative count, unknown enum value, bad handle */
    ISO_ERR_DIMS = 2,    /* d outside 1..ISO_MAX_DIMS, a dimension size < 1, P too large */
    ISO_ERR_COUNT = 3,   /* send and receive block sizes differ, or a size overflows */
    ISO_ERR_ALIGN = 4,   /* reserved: no supported input is rejected for alignment */
    ISO_ERR_NOMEM = 5,   /* host or device allocation failed */
    ISO_ERR_CUDA = 6,    /* a CUDA call failed; see Iso_last_cuda_error */
    ISO_ERR_OVERLAP = 7, /* receive blocks overlap each other, or send and receive buffers overlap */
    ISO_ERR_STATE = 8,   /* call not valid in this state (e.g. request bound to no buffers) */
    ISO_ERR_TIMEOUT = 9, /* a bounded wait inside a kernel expired; the result is incomplete */
    ISO_ERR_TOO_LARGE = 10 /* Iso_neighbor_alltoall_static: tables + intermediate buffer exceed
                              ISO_STATIC_SCRATCH_BYTES */
};

/* Schedules. */
enum {
    ISO_ALG_COMBINING = 0, /* Section V: message combining with direct communication along
                              the dimensions, one round per distinct non-zero coordinate */
    ISO_ALG_DIRECT = 1,    /* Listing 3: every block straight from its source, here in one pass */
    ISO_ALG_TORUS = 2      /* Section III, Algorithm 1: hop-by-hop between immediate neighbours */
};

/* Where the message-combining all-to-all keeps a block between two hops. */
enum {
    ISO_LAYOUT_PACKED = 0,      /* every non-final hop has its own place in the intermediate buffer,
                                   places ordered by (writing phase, reading phase, neighbour) so that
                                   a phase touches few contiguous regions; receive buffer written by
                                   final hops only.  Intermediate buffer: sum_i (hops_i - 1) blocks */
    ISO_LAYOUT_ALTERNATING = 1  /* Algorithm 1: the block alternates between its slot of the receive
                                   buffer and its slot of an equally large intermediate buffer */
};

enum { ISO_KIND_ALLTOALL = 0, ISO_KIND_ALLGATHER = 1, ISO_KIND_ALLTOALLV = 2 };
enum { ISO_BUF_SEND = 0, ISO_BUF_RECV = 1, ISO_BUF_INTER = 2 };

typedef struct Iso_stats {
    int kind;             /* ISO_KIND_* */
    int algorithm;        /* ISO_ALG_* */
    int fusion_level;
    int d;
    int s;
    int rounds;           /* communication rounds of the schedule (Sections III-A and V) */
    int max_rounds_per_dim; /* the factor N of the paper's N*d bound on the rounds */
    int phases;           /* groups of rounds that run without an ordering point between them */
    int launches;         /* kernel launches per Iso_Start */
    int parts;            /* block transmissions per process: sum of hops (all-to-all),
                             trie edges that move a block (allgather) */
    int local_copies;     /* blocks whose source is the process itself (no hop) */
    int64_t P;
    int64_t send_stride;  /* bytes between consecutive processes' send buffers */
    int64_t recv_stride;
    int64_t inter_stride; /* same for the library's intermediate buffer (0: none needed) */
    int64_t bytes_min;    /* 2 * P * sum_i m_i: every delivered block read once, written once */
    int64_t bytes_moved;  /* bytes read + written by one Iso_Start with this schedule as it is
                             lowered (an allgather phase in sender-side form reads a block once for
                             up to four copies) */
    int64_t bulk_bytes;   /* part of bytes_moved handled by the bulk-copy kernel */
} Iso_stats;

/* One line of a schedule as it is executed: in phase `phase`, every process r copies
 * `len` bytes from byte `src_off` of buffer `src_buf` of process r (-) shift to byte
 * `dst_off` of its own buffer `dst_buf`.  `slot` is the neighbour index i the bytes belong
 * to; `round` numbers the paper's communication rounds (-1 for a local copy). */
typedef struct Iso_part {
    int phase;
    int round;
    int slot;
    int src_buf;          /* ISO_BUF_* */
    int dst_buf;
    int kernel;           /* 0: vector copy kernel, 1: bulk copy kernel, 2: vector copy kernel in its
                             sender-side form (allgather phases: a block is loaded once and stored
                             to every place it is copied to) */
    int width;            /* bytes per vector unit (vector kernel) */
    int reserved;
    int64_t src_off;
    int64_t dst_off;
    int64_t len;
    int shift[ISO_MAX_DIMS]; /* per dimension, reduced to [0, p_j); signed on non-periodic dimensions */
    int check[ISO_MAX_DIMS]; /* non-periodic dimensions: process x takes part only if
                                0 <= x_j - check_j < p_j (0: no condition) */
} Iso_part;

/*
 * Neighbourhood set-up (Listing 1, Section II).  `dims[0..d-1]` are the torus sizes,
 * `relative_coordinates` holds s*d integers, neighbour-major (vector i occupies entries
 * i*d .. i*d+d-1).  Any integers are allowed: repetitions, the zero vector, coordinates
 * whose magnitude exceeds the torus size.  The order of the vectors fixes the order of
 * the blocks in the buffers.  s = 0 is valid.  The arrays are copied.
 * Errors: ISO_ERR_ARG (null pointer, s < 0), ISO_ERR_DIMS, ISO_ERR_NOMEM.
 */
int Iso_neighborhood_create(int d, const int dims[], int s, const int relative_coordinates[],
                            Iso_comm *isocomm);

/* Releases the neighbourhood; requests created from it keep it alive until they are freed.
 * `*isocomm` is set to NULL. */
int Iso_comm_free(Iso_comm *isocomm);

/*
 * Regular all-to-all (Listing 2, Section II): s blocks of sendcount * sendtype bytes per
 * process, stored consecutively in neighbour order in both buffers.  The block sizes in
 * bytes on the send and receive side must be equal (ISO_ERR_COUNT otherwise).
 * The schedule (Section V with the buffer alternation of Algorithm 1) is computed here, on
 * the host; device resources (the intermediate buffer and the index tables) are created by
 * the first Iso_Start.  `sendbuf` and `recvbuf` are device pointers owned by the caller,
 * must not overlap, must stay valid while the request is in use; the send buffer is never
 * written.  Both may be NULL: the request can then be inspected (statistics, parts) but
 * not started.
 */
int Iso_neighbor_alltoall_init(const void *sendbuf, int sendcount, Iso_datatype sendtype,
                               void *recvbuf, int recvcount, Iso_datatype recvtype,
                               Iso_comm isocomm, Iso_request *request);

/*
 * Allgather (Listing 2, Sections II and III-B): every process contributes ONE block of
 * sendcount * sendtype bytes and receives s blocks in neighbour order.  The schedule is
 * the prefix-trie schedule of Section III-B in its direct-communication form (Section V).
 * Buffer rules as for the all-to-all.
 */
int Iso_neighbor_allgather_init(const void *sendbuf, int sendcount, Iso_datatype sendtype,
                                void *recvbuf, int recvcount, Iso_datatype recvtype,
                                Iso_comm isocomm, Iso_request *request);

/*
 * Irregular all-to-all (Listing 4, Section II): block i has sendcounts[i] elements at
 * byte displacement senddispls[i] of a process's send buffer and arrives at byte
 * displacement recvdispls[i] of the receiver's buffer.  Counts and displacements (s
 * entries each, host arrays, copied) are the same on every process and block sizes must
 * match pairwise in bytes (ISO_ERR_COUNT).  Displacements must be >= 0; receive blocks
 * must not overlap each other (ISO_ERR_OVERLAP); send blocks may.  The schedules are those
 * of the regular case (Section IV).
 */
int Iso_neighbor_alltoallv_init(const void *sendbuf, const int sendcounts[],
                                const int64_t senddispls[], Iso_datatype sendtype,
                                void *recvbuf, const int recvcounts[],
                                const int64_t recvdispls[], Iso_datatype recvtype,
                                Iso_comm isocomm, Iso_request *request);

/*
 * Irregular allgather (Listing 4): one send block of sendcount * sendtype bytes per
 * process; the copy received from neighbour i is stored at byte displacement
 * recvdispls[i]; recvcounts[i] * recvtype must equal the send block size for every i.
 */
int Iso_neighbor_allgatherv_init(const void *sendbuf, int sendcount, Iso_datatype sendtype,
                                 void *recvbuf, const int recvcounts[],
                                 const int64_t recvdispls[], Iso_datatype recvtype,
                                 Iso_comm isocomm, Iso_request *request);

/*
 * Chooses the schedule.  `alg` is an ISO_ALG_* value.  `fusion_level` applies to
 * ISO_ALG_COMBINING: 0 = one kernel launch per communication round; 1 (the default) = all
 * rounds of one dimension in one launch (same bytes moved: within a dimension every block
 * moves at most once); g >= 2 = the dimensions are taken in groups of g consecutive ones and
 * a block's hops inside a group are composed into a single shift (Section V combines all
 * blocks bound for the same relative neighbour), so fewer intermediate copies
 * pass through memory; g >= d moves exactly the bytes of ISO_ALG_DIRECT.
 * May be called at any time between starts; the schedule is rebuilt and the device tables
 * are replaced by the next Iso_Start.  Errors: ISO_ERR_ARG.
 */
int Iso_request_set_algorithm(Iso_request request, int alg, int fusion_level);

/* Chooses the intermediate-storage layout (ISO_LAYOUT_*) of ISO_ALG_COMBINING all-to-all
 * schedules; the hop-by-hop schedule always alternates as in Algorithm 1.  Default: packed. */
int Iso_request_set_layout(Iso_request request, int layout);

/*
 * One-launch execution.  When every launch of the schedule is a 16-byte vector launch on
 * periodic dimensions, Iso_Start runs all phases in ONE cooperative kernel launch: the
 * thread blocks go through the phases together and meet at a grid-wide barrier between
 * them (the ordering point the paper gets from completing a round's MPI_Sendrecv), which
 * saves the ramp-up and drain of one kernel per phase.  The barrier wait is bounded; if it
 * expires the kernel stops and Iso_wait returns ISO_ERR_TIMEOUT.  enable = 0 goes back to
 * one launch per phase, which is the default: with programmatic dependent launches between
 * the phases the per-phase kernels are faster (36.1 against 44.9 microseconds on the 32^3
 * torus, 161 against 197 microseconds on the 8^5 torus with five phases).  Iso_request_get_stats
 * reports launches = 1 once the request has been started in this mode.
 */
int Iso_request_set_single_launch(Iso_request request, int enable);

/*
 * Pipelined one-launch execution (no counterpart in the paper).  `slabs` >= 1 makes Iso_Start
 * a single cooperative kernel launch that needs no grid-wide barrier: the torus is cut into
 * `slabs` slabs of consecutive planes of dimension 0 (as for Iso_request_set_slabs, under the
 * same condition; 1, or a schedule that cannot be cut, means the whole torus) and the work
 * into items (slab, launch of the schedule).  All thread blocks go through the items in one
 * order - the launches of two slabs interleaved - and every item has a counter of the thread
 * blocks that have finished it; a block starts an item when the item it depends on (the
 * same slab's previous phase, or the last reader of the intermediate place it overwrites) is
 * complete, which in that order has normally happened already.  A slab's intermediate blocks
 * are read back out of the L2 cache a few items after they were written, and from three
 * slabs on the intermediate buffer holds only two slabs.  Requires what the single launch
 * requires (16-byte vector launches on periodic dimensions: blocks that are multiples of
 * 16 bytes and below the bulk threshold, or Iso_request_set_bulk_threshold(request, 0));
 * where that does not hold the request runs as if this had not been called.  It takes
 * precedence over Iso_request_set_single_launch, _set_slabs, _set_chains and _set_graph, and
 * Iso_request_tune leaves such a request alone.  Every wait is bounded; on expiry the
 * kernel stops and Iso_wait returns ISO_ERR_TIMEOUT.  0 (default) turns it off.  The result
 * never depends on it.
 */
int Iso_request_set_pipeline(Iso_request request, int slabs);

/*
 * Slab execution.  When only blocks read from the send buffer move along dimension 0 (the
 * combining and direct schedules on periodic tori) the torus can be processed in slabs of
 * consecutive planes of dimension 0, all phases of one slab before the next slab: a slab's
 * intermediate blocks are then read back while still in the L2 cache, and the intermediate
 * buffer only holds one slab and is reused, so its lines are overwritten in cache instead of
 * being written to device memory.  `slabs` = 0 (default) lets the library choose (vector
 * launches only, and only when a slab's launch still lasts about 12 microseconds), 1 turns
 * it off, n >= 2 asks for n slabs (at most the size of dimension 0; ignored when the
 * schedule does not allow it or in single-launch mode).  The result never depends on it.
 */
int Iso_request_set_slabs(Iso_request request, int slabs);

/*
 * Slabs side by side (no counterpart in the paper).  With `chains` = n >= 2 the slabs of
 * Iso_request_set_slabs are dealt to n chains that run at the same time, each on 1/n of
 * the CTA slots and with its own one-slab part of the intermediate buffer: the start and
 * the drain of one chain's short kernels are covered by the other chains.  The number of
 * slabs is rounded to a multiple of n; the launches are then replayed from a captured
 * graph (see Iso_request_set_graph).  1 (default) turns it off; at most 8.  Ignored where
 * slab execution is (see there).  The result never depends on it.
 */
int Iso_request_set_chains(Iso_request request, int chains);

/*
 * Graph replay (no counterpart in the paper).  With `enable` != 0 the first Iso_Start after
 * a change of the request captures its launches into a CUDA graph on a stream of the
 * library's own and every Iso_Start replays that graph on the caller's stream: one
 * submission per start instead of one per launch, which pays for schedules of many short
 * launches and costs a few microseconds on schedules of few long ones.  With `enable` == 0
 * (the default) the library replays from a graph only where a start has 128 launches or
 * more.  Ignored in single-launch mode.  The result never depends on it.
 */
int Iso_request_set_graph(Iso_request request, int enable);

/*
 * Measures instead of guessing (no counterpart in the paper; in the spirit of its
 * persistent requests, which are set up once and started many times): runs the request
 * with 1, 2, 4, ... slabs, with 1, 2 and 4 chains, with and without graph replay (and, for
 * ragged rows, with and without the bulk warps of Iso_request_set_hybrid), timing a
 * few starts of each on `cuda_stream` with events, and leaves the request on the fastest
 * combination (a less plain plan has to win by 2 %).  `flags` is a sum of ISO_TUNE_* values.
 * Without ISO_TUNE_COLD the starts are timed back to back, as in a loop over the same
 * buffers; with it a scratch buffer of twice the L2 size is overwritten before every timed
 * start (allocated for the duration of the call), as when other work runs between the
 * starts.  With ISO_TUNE_SCHEDULE the schedule is chosen as well: the message-combining
 * schedule with one and with two dimensions per phase (for an allgather in both visiting
 * orders of the dimensions, see Iso_request_set_dimension_order) and the direct schedule are
 * all timed, each under every execution plan, and the request is left on the fastest (on one device
 * the direct schedule usually wins: it moves the fewest bytes); Iso_request_get_stats then
 * reports the algorithm and fusion level in use, Iso_request_get_execution the plan.
 * Without it the request keeps its schedule.  The collective is executed many times meanwhile:
 * the send buffers must hold readable data and the receive buffers are overwritten (with
 * the collective's result).  Blocks the host until done.  Does nothing in single-launch
 * mode.  On error the settings from before the call are restored.
 */
enum { ISO_TUNE_COLD = 1, ISO_TUNE_SCHEDULE = 2 };
int Iso_request_tune(Iso_request request, void *cuda_stream, int flags);

/* What Iso_Start does at present: slabs (1: none), chains (1: none), graph replay (0/1).
 * Before the first Iso_Start after a change these are the values asked for (slabs 0:
 * automatic); any of the pointers may be NULL. */
int Iso_request_get_execution(Iso_request request, int *slabs, int *chains, int *graph);

/*
 * Ragged rows of the irregular collectives (no counterpart in the paper).  A launch whose
 * pieces need several unit widths normally moves everything through the vector kernel.  With
 * `enable` != 0 the 16-byte-aligned bodies of at least 256 bytes among its pieces are moved
 * by bulk copies instead, issued by extra warps of the same thread blocks while the other
 * warps move the short pieces and ragged ends (up to three dimensions, periodic, bulk
 * threshold not 0).  Measured on irregular sizes from {4, ..., 1024} bytes: 22 % faster for the
 * one-pass direct schedule on the 64x64x32 torus, 15 % slower for the combining schedule in
 * slabs, hence off by default; Iso_request_tune tries both.  The result never depends on it.
 */
int Iso_request_set_hybrid(Iso_request request, int enable);

/*
 * Sender-side form of allgather phases (Section III-B: a block travels once per trie edge).
 * A phase of the allgather schedules copies one block to several places; run as a gather,
 * every copy loads the block again.  In sender-side form a thread loads a 16-byte unit of
 * the block once, from the process that holds it, and stores it to up to four of its
 * destinations (a block with more copies is loaded once per four).  mode 0: never;
 * 1 (default): in the phases where it measured faster (no block with more than four copies,
 * at least 64 MiB written); 2: in every phase that allows it - blocks that are multiples of
 * 16 bytes and below the bulk threshold, one shifted dimension per phase, periodic, no slab,
 * chain or one-launch execution asked for.  The result never depends on it;
 * Iso_request_get_stats counts a block read once per load in bytes_moved.
 */
int Iso_request_set_sender_side(Iso_request request, int mode);

/* Allgather, message-combining schedule: the order in which the prefix trie visits the
 * dimensions (Section III-B leaves it open; the received data never depends on it, the number
 * of parts may for neighbourhoods that are not symmetric in the dimensions).  order[k] is the
 * dimension visited k-th, a permutation of 0..d-1 (host array, read during the call).  Stored
 * for the other collectives but without effect there.  Rebuilds the schedule; waits for a
 * start in flight first.  ISO_ERR_ARG if `order` is not a permutation. */
int Iso_request_set_dimension_order(Iso_request request, const int order[]);
/* The order in use: d values written to `order` (host array).  Default for the allgather:
 * last dimension first when the neighbours have at most 8 distinct non-zero coordinates in
 * dimension 0 (the last phase then copies runs of consecutive receive slots), first to last
 * otherwise; 0..d-1 for the other collectives. */
int Iso_request_get_dimension_order(Iso_request request, int order[]);

/* Parts of at least `bytes` bytes whose addresses and length are multiples of 16 are moved
 * by the bulk-copy kernel (asynchronous bulk copies staged through shared memory), the rest
 * by the vector kernel.  Left to the library (no call, the default): 512 - measured crossover
 * of one launch against one launch - except for an all-to-all with intermediate blocks whose
 * slab count is also left to the library (Iso_request_set_slabs), where it is 4096: the vector
 * kernel in slabs, whose intermediate blocks are read back out of the L2, measured 5 to 12 %
 * faster than the bulk kernel on 512-byte to 2 KB blocks and 11 % slower on 4 KB blocks.
 * 0 disables the bulk kernel. */
int Iso_request_set_bulk_threshold(Iso_request request, int64_t bytes);

/*
 * Non-periodic dimensions (the extension Section VII mentions).  periodic[j] = 0 makes
 * dimension j a mesh: a block whose source R - C^i falls outside the mesh is not delivered
 * and the receive slot keeps its previous contents.  Supported by ISO_ALG_DIRECT and by
 * ISO_ALG_COMBINING for all collectives.  All-to-all: every hop of a block is skipped for
 * the processes on whose route the original sender or the final receiver would lie outside
 * (always with the packed layout: the receive buffer cannot double as scratch when
 * undelivered slots must keep their contents).  Allgather: a trie node is produced only at
 * the processes whose source for that prefix exists.  ISO_ALG_TORUS (Algorithm 1 as
 * printed, whose blocks alternate through their receive slots) is refused with ISO_ERR_ARG.
 * Call it before creating requests.  Default: all dimensions periodic.
 */
int Iso_comm_set_periodic(Iso_comm isocomm, const int periodic[]);

/*
 * Runs the collective: enqueues the schedule's kernels on `cuda_stream` (a cudaStream_t
 * cast to void*, NULL = the default stream) and returns without waiting (the non-blocking
 * start proposed in Section VII).  The first start after an init or a set_* call also
 * allocates the intermediate buffer and uploads the index tables (cudaMalloc and a blocking
 * copy), so it must not happen inside a stream capture.  Starts of one request are ordered
 * by the stream they are enqueued on: a request owns one intermediate buffer, so two starts
 * of the same request on different streams must not overlap.
 * Errors: ISO_ERR_STATE (request has no buffers), ISO_ERR_NOMEM, ISO_ERR_CUDA.
 */
int Iso_Start(Iso_request request, void *cuda_stream);

/* Same with HOST buffers holding all P processes' send / receive buffers in the layout
 * above: copies `host_sendbuf` to the request's device send buffer, runs the schedule and
 * copies the device receive buffer to `host_recvbuf`.  When only blocks read from the send
 * buffer move along dimension 0 (true for the combining and direct schedules on periodic
 * tori with at least four planes) the work is pipelined over up to 32 slabs of
 * dimension 0: a slab's schedule runs as soon as the slabs it reads from have arrived and
 * its receive buffers travel back while later slabs are still being uploaded (uploads and
 * downloads on two internal streams created by the first such call, kernels on
 * `cuda_stream`, which is made to wait for the downloads).  Otherwise: one upload, the
 * schedule, one download, all on `cuda_stream`.  The copies are asynchronous when the host
 * memory is page-locked.  Complete after Iso_wait or a synchronisation of `cuda_stream`. */
int Iso_Start_host(Iso_request request, const void *host_sendbuf, void *host_recvbuf,
                   void *cuda_stream);

/*
 * Link-busy times of the last pipelined Iso_Start_host of this request (measurement aid):
 * milliseconds between the first upload starting and the last one ending, the same for the
 * downloads, and for the whole call on `cuda_stream`; `slabs` = slabs it was pipelined over.
 * Any pointer may be NULL.  Waits for the request first.  ISO_ERR_STATE when the last start
 * was not a pipelined Iso_Start_host.
 */
int Iso_request_get_host_transfer_ms(Iso_request request, float *upload_ms, float *download_ms, float *total_ms,
                                     int *slabs);

/* Local completion (Section VII): blocks until the last start has finished and returns
 * ISO_ERR_TIMEOUT if a kernel gave up a bounded wait, ISO_ERR_CUDA on a CUDA error.
 * After ISO_ERR_TIMEOUT the receive buffers are incomplete, the request's arrival counters
 * have been cleared and the request can be started again. */
int Iso_wait(Iso_request request);

/*
 * Race detection aid (no counterpart in the paper).  The library's intermediate buffer is
 * allocated with a guard band of 4096 bytes of a fixed pattern on either side; a schedule
 * never writes there.  This call waits for the request's work in flight, reads both bands
 * back and stores the number of bytes that no longer hold the pattern in `*violations`
 * (0 when the request has no intermediate buffer yet).  Meant for tests, together with
 * bands the caller puts around its own send and receive buffers.
 */
int Iso_request_check_guards(Iso_request request, int64_t *violations);

/*
 * Bound of the device-side waits (no counterpart in the paper, whose processes block in
 * MPI_Sendrecv).  The one-launch execution modes (Iso_request_set_single_launch,
 * Iso_request_set_pipeline) make thread blocks wait for each other; every such wait polls
 * at most `polls` times (about 40 ns apart) and then gives up: the kernel returns by itself
 * and Iso_wait reports ISO_ERR_TIMEOUT.  Default 2^22 (a fraction of a second).  polls >= 1.
 */
int Iso_request_set_wait_limit(Iso_request request, unsigned int polls);

/*
 * Testing aid for the time-out path.  The NEXT start of a one-launch execution mode waits
 * for `extra` more arrivals than there are thread blocks, so its first wait cannot be
 * satisfied and runs into the limit set with Iso_request_set_wait_limit; nothing faults
 * and nothing waits without bound.  One shot: later starts are normal.  0 <= extra <= 1024.
 * Has no effect on the default execution (one launch per phase), which has no such waits.
 */
int Iso_request_test_skew_arrivals(Iso_request request, int extra);

/*
 * Launch-latency floor (measurement aid, no counterpart in the paper): enqueues `launches`
 * launches of an empty kernel back to back on `cuda_stream`, as programmatic dependent
 * launches when `dependent` != 0 (the way Iso_Start chains its phases), times them with
 * events and stores the device time per launch in microseconds.  Blocks until done.
 * A phase of a schedule cannot be shorter than this.
 */
int Iso_measure_launch_floor(void *cuda_stream, int launches, int dependent, float *microseconds_per_launch);

/* Statistics of the current schedule.  Host only; valid before the first start. */
int Iso_request_get_stats(Iso_request request, Iso_stats *out);

/* Copies up to `capacity` executed parts (in execution order) to `out` and stores the
 * total number in `*count`.  Needs no device; meant for validation of schedules. */
int Iso_request_get_parts(Iso_request request, Iso_part *out, int capacity, int *count);

/*
 * Regular message-combining all-to-all that allocates no device memory.  (The paper has no
 * counterpart: its library may allocate freely inside the init call.)
 *
 * For callers that cannot allocate where they need the collective: programs whose device
 * memory was budgeted and handed out at start-up, plug-ins living inside another
 * framework's memory pool, hot paths where a cudaMalloc - which synchronises the device -
 * is not acceptable.  Iso_neighbor_alltoall_init / Iso_Start keep their unit tables and
 * their intermediate buffer in memory obtained with cudaMalloc; this call keeps both in a
 * fixed scratch array of ISO_STATIC_SCRATCH_BYTES bytes that is part of the library image
 * (every device that loads the library holds one copy until the process exits) and calls
 * no cudaMalloc, cudaFree, cudaMallocHost or other allocating CUDA routine.  The schedule
 * itself is computed on the host with ordinary heap memory that is released before return.
 *
 * Same arguments as Iso_neighborhood_create + Iso_neighbor_alltoall_init (send and receive
 * blocks of count * type bytes, both buffers DEVICE pointers owned by the caller, layout
 * as described at the top of this file) plus the stream; the schedule is ISO_ALG_COMBINING,
 * one launch per dimension, packed layout, vector kernel only.  The call copies the tables
 * into the scratch area and enqueues the kernels on `cuda_stream`; it does not wait.
 *
 * Limits and rules:
 *  - P * (intermediate bytes per process) + the unit tables must fit the scratch array,
 *    else ISO_ERR_TOO_LARGE and nothing is enqueued;
 *  - the first call on a device looks up the device address of the scratch array
 *    (cudaGetSymbolAddress, with that device current);
 *  - NO call of this function, first or later, may be made while `cuda_stream` is being
 *    captured into a graph: every call copies freshly built tables from host memory that
 *    is released when the call returns, so a captured copy node would read freed memory
 *    at every replay;
 *  - all calls on one device share the scratch array and it keeps the previous call's
 *    contents; nothing in it has to start at zero, because every byte a kernel reads from
 *    it was written earlier in the same call (tables by the copy, intermediate places by
 *    an earlier phase).  Two calls whose work overlaps on the GPU (different streams, or
 *    different host threads) race on it: keep calls on one device in one stream order.
 * Errors: ISO_ERR_ARG, ISO_ERR_DIMS, ISO_ERR_COUNT, ISO_ERR_OVERLAP, ISO_ERR_TOO_LARGE,
 * ISO_ERR_CUDA.
 */
#define ISO_STATIC_SCRATCH_BYTES (8u << 20)
int Iso_neighbor_alltoall_static(int d, const int dims[], int s, const int relative_coordinates[],
                                 const void *sendbuf, void *recvbuf, int count, Iso_datatype type,
                                 void *cuda_stream);

/* Frees the request, its device memory and its reference on the neighbourhood; waits for
 * work in flight first.  `*request` is set to NULL. */
int Iso_request_free(Iso_request *request);

/* Static text for an ISO_ERR_* code. */
const char *Iso_error_string(int code);

/* The cudaError_t value of the CUDA call that last failed inside the library on this
 * host thread (0 if none). */
int Iso_last_cuda_error(void);

/* Host-side consistency checks of the library's integer helpers (exact division by
 * multiplication, alignment classes).  Returns ISO_SUCCESS or ISO_ERR_STATE.  No device. */
int Iso_selftest(void);

#ifdef __cplusplus
}
#endif
#endif /* ISO_H */
