/*
 * CPU oracle for isomorphic, sparse neighbourhood collectives on a d-dimensional
 * periodic torus.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain definition of the result,
 * written for checking by eye against the paper; it is slow on purpose, shares
 * no code with the CUDA library and must never be called from the product path.
 *
 * Definitions followed (paper, Section II):
 *   - p processes in a torus with sizes p_0..p_{d-1}; process R has coordinates
 *     (r_0..r_{d-1}), 0 <= r_j < p_j.
 *   - an s-neighbourhood is an ordered list of s integer offset vectors C^i
 *     (repetitions, the zero vector and |c| >= p_j all allowed).
 *   - torus addition: R (+) C = ((r_j + c_j) mod p_j)_j.  Process R sends block i
 *     to R (+) C^i and therefore receives block i from R (-) C^i.
 *   - blocks sit consecutively in the send / receive buffer in neighbour order.
 *   - all-to-all: an individual block per neighbour; allgather: the same single
 *     block to every neighbour; irregular all-to-all: block i has its own length
 *     and byte displacement, identical on every process.
 *
 * The paper leaves the rank <-> coordinate mapping to the Cartesian communicator;
 * the reading used here is row-major with dimension d-1 varying fastest.
 *
 * All P processes' buffers are stored process-major: process q's buffer starts
 * at byte q * stride.  Every function computes the receive buffers of the
 * destination ranks r0 <= r < r1 only, and `recv` points at the first byte of
 * rank r0's receive buffer, so that large cases can be produced in chunks.
 *
 * Return value: 0 on success, -1 on an invalid argument.
 */
#include <stdint.h>
#include <string.h>

#define ISO_ORACLE_MAX_DIMS 16

/* Rank of the process at coordinates R (-) C, where R are the coordinates of
 * rank r.  Section II: component-wise subtraction modulo p_j. */
int64_t iso_oracle_source_rank(int d, const int *dims, int64_t r, const int *C)
{
    int64_t coord[ISO_ORACLE_MAX_DIMS];
    int64_t rest = r;
    int j;
    /* rank -> coordinates, dimension d-1 fastest */
    for (j = d - 1; j >= 0; j--) {
        coord[j] = rest % dims[j];
        rest = rest / dims[j];
    }
    /* R (-) C */
    for (j = 0; j < d; j++) {
        int64_t p = dims[j];
        int64_t x = (coord[j] - (int64_t)C[j]) % p;
        if (x < 0)
            x += p;
        coord[j] = x;
    }
    /* coordinates -> rank */
    rest = 0;
    for (j = 0; j < d; j++)
        rest = rest * dims[j] + coord[j];
    return rest;
}

/* Rank of the process at R (+) C (the target of a send); used by tests that
 * state the collective from the sender's side. */
int64_t iso_oracle_target_rank(int d, const int *dims, int64_t r, const int *C)
{
    int neg[ISO_ORACLE_MAX_DIMS];
    int j;
    for (j = 0; j < d; j++)
        neg[j] = -C[j];
    return iso_oracle_source_rank(d, dims, r, neg);
}

static int args_ok(int d, const int *dims, int s, int64_t r0, int64_t r1)
{
    int64_t P = 1;
    int j;
    if (d < 1 || d > ISO_ORACLE_MAX_DIMS || s < 0 || dims == 0)
        return 0;
    for (j = 0; j < d; j++) {
        if (dims[j] < 1)
            return 0;
        P *= dims[j];
    }
    return 0 <= r0 && r0 <= r1 && r1 <= P;
}

/* Regular all-to-all, blocks of m bytes:
 *   recv[r][i] = send[rank(R (-) C^i)][i]        for every r, i. */
int iso_oracle_alltoall(int d, const int *dims, int s, const int *offsets,
                        int64_t m, const unsigned char *send, unsigned char *recv,
                        int64_t r0, int64_t r1)
{
    int64_t r;
    int i;
    if (!args_ok(d, dims, s, r0, r1) || m < 0)
        return -1;
    for (r = r0; r < r1; r++) {
        for (i = 0; i < s; i++) {
            int64_t q = iso_oracle_source_rank(d, dims, r, offsets + (int64_t)i * d);
            memcpy(recv + ((r - r0) * s + i) * m, send + (q * s + i) * m, (size_t)m);
        }
    }
    return 0;
}

/* Allgather, one block of m bytes per process:
 *   recv[r][i] = send[rank(R (-) C^i)]           for every r, i. */
int iso_oracle_allgather(int d, const int *dims, int s, const int *offsets,
                         int64_t m, const unsigned char *send, unsigned char *recv,
                         int64_t r0, int64_t r1)
{
    int64_t r;
    int i;
    if (!args_ok(d, dims, s, r0, r1) || m < 0)
        return -1;
    for (r = r0; r < r1; r++) {
        for (i = 0; i < s; i++) {
            int64_t q = iso_oracle_source_rank(d, dims, r, offsets + (int64_t)i * d);
            memcpy(recv + ((r - r0) * s + i) * m, send + q * m, (size_t)m);
        }
    }
    return 0;
}

/* Irregular all-to-all: block i has len[i] bytes, lies at byte sdispl[i] of a
 * process's send buffer and arrives at byte rdispl[i] of the receiver's buffer;
 * lengths and displacements are the same on every process.  Process q's send
 * buffer starts at q * send_stride, its receive buffer at q * recv_stride.
 *   recv[r] + rdispl[i] .. + len[i]  =  send[rank(R (-) C^i)] + sdispl[i] .. */
int iso_oracle_alltoallv(int d, const int *dims, int s, const int *offsets,
                         const int64_t *len, const int64_t *sdispl, const int64_t *rdispl,
                         int64_t send_stride, int64_t recv_stride,
                         const unsigned char *send, unsigned char *recv,
                         int64_t r0, int64_t r1)
{
    int64_t r;
    int i;
    if (!args_ok(d, dims, s, r0, r1))
        return -1;
    for (i = 0; i < s; i++)
        if (len[i] < 0 || sdispl[i] < 0 || rdispl[i] < 0)
            return -1;
    for (r = r0; r < r1; r++) {
        for (i = 0; i < s; i++) {
            int64_t q = iso_oracle_source_rank(d, dims, r, offsets + (int64_t)i * d);
            memcpy(recv + (r - r0) * recv_stride + rdispl[i],
                   send + q * send_stride + sdispl[i], (size_t)len[i]);
        }
    }
    return 0;
}

/* ---- non-periodic (mesh) dimensions ------------------------------------------------
 *
 * Section VII of the paper mentions the extension to tori in which some dimensions do
 * not wrap around.  Reading used here: along a dimension j with periodic[j] == 0 the
 * coordinates are not reduced; process R receives block i only if its source R - C^i
 * exists, i.e. 0 <= r_j - c_j < p_j in every such dimension.  Otherwise nothing is
 * delivered and the receive slot keeps whatever it held before the call.  Periodic
 * dimensions wrap as above.
 *
 * Returns the source rank, or -1 when the source lies outside the mesh. */
int64_t iso_oracle_source_rank_mesh(int d, const int *dims, const int *periodic, int64_t r, const int *C)
{
    int64_t coord[ISO_ORACLE_MAX_DIMS];
    int64_t rest = r;
    int j;
    for (j = d - 1; j >= 0; j--) {
        coord[j] = rest % dims[j];
        rest = rest / dims[j];
    }
    for (j = 0; j < d; j++) {
        int64_t p = dims[j];
        int64_t y = coord[j] - (int64_t)C[j];
        if (periodic[j]) {
            y = y % p;
            if (y < 0)
                y += p;
        } else if (y < 0 || y >= p) {
            return -1;
        }
        coord[j] = y;
    }
    rest = 0;
    for (j = 0; j < d; j++)
        rest = rest * dims[j] + coord[j];
    return rest;
}

/* All-to-all on a mesh: recv[r][i] = send[R - C^i][i] where that process exists;
 * other slots of `recv` are left as they are. */
int iso_oracle_alltoall_mesh(int d, const int *dims, const int *periodic, int s, const int *offsets,
                             int64_t m, const unsigned char *send, unsigned char *recv,
                             int64_t r0, int64_t r1)
{
    int64_t r;
    int i;
    if (!args_ok(d, dims, s, r0, r1) || m < 0 || periodic == 0)
        return -1;
    for (r = r0; r < r1; r++) {
        for (i = 0; i < s; i++) {
            int64_t q = iso_oracle_source_rank_mesh(d, dims, periodic, r, offsets + (int64_t)i * d);
            if (q < 0)
                continue;
            memcpy(recv + ((r - r0) * s + i) * m, send + (q * s + i) * m, (size_t)m);
        }
    }
    return 0;
}

/* Allgather on a mesh: recv[r][i] = send[R - C^i] where that process exists. */
int iso_oracle_allgather_mesh(int d, const int *dims, const int *periodic, int s, const int *offsets,
                              int64_t m, const unsigned char *send, unsigned char *recv,
                              int64_t r0, int64_t r1)
{
    int64_t r;
    int i;
    if (!args_ok(d, dims, s, r0, r1) || m < 0 || periodic == 0)
        return -1;
    for (r = r0; r < r1; r++) {
        for (i = 0; i < s; i++) {
            int64_t q = iso_oracle_source_rank_mesh(d, dims, periodic, r, offsets + (int64_t)i * d);
            if (q < 0)
                continue;
            memcpy(recv + ((r - r0) * s + i) * m, send + q * m, (size_t)m);
        }
    }
    return 0;
}

/* Irregular all-to-all on a mesh. */
int iso_oracle_alltoallv_mesh(int d, const int *dims, const int *periodic, int s, const int *offsets,
                              const int64_t *len, const int64_t *sdispl, const int64_t *rdispl,
                              int64_t send_stride, int64_t recv_stride,
                              const unsigned char *send, unsigned char *recv,
                              int64_t r0, int64_t r1)
{
    int64_t r;
    int i;
    if (!args_ok(d, dims, s, r0, r1) || periodic == 0)
        return -1;
    for (i = 0; i < s; i++)
        if (len[i] < 0 || sdispl[i] < 0 || rdispl[i] < 0)
            return -1;
    for (r = r0; r < r1; r++) {
        for (i = 0; i < s; i++) {
            int64_t q = iso_oracle_source_rank_mesh(d, dims, periodic, r, offsets + (int64_t)i * d);
            if (q < 0)
                continue;
            memcpy(recv + (r - r0) * recv_stride + rdispl[i],
                   send + q * send_stride + sdispl[i], (size_t)len[i]);
        }
    }
    return 0;
}
