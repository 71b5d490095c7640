/* A plain C program against include/iso.h: proves that the header is valid C and that the
 * host-side entry points work without Python and without a GPU. */
#include <stdio.h>
#include <string.h>

#include "iso.h"

#define CHECK(cond)                                                        \
    do {                                                                   \
        if (!(cond)) {                                                     \
            printf("FAILED line %d: %s\n", __LINE__, #cond);               \
            return 1;                                                      \
        }                                                                  \
    } while (0)

int main(void)
{
    /* the positive-octant example of Section II of the paper: 7 neighbours in 3 dimensions */
    int dims[3] = {6, 5, 4};
    int octant[] = {1, 0, 0, 0, 1, 0, 0, 0, 1, 1, 1, 0, 1, 0, 1, 0, 1, 1, 1, 1, 1};
    Iso_comm comm = NULL;
    Iso_request req = NULL;
    Iso_stats st;
    Iso_part parts[64];
    int count = 0, i;

    CHECK(Iso_selftest() == ISO_SUCCESS);
    CHECK(Iso_neighborhood_create(3, dims, 7, octant, &comm) == ISO_SUCCESS);
    CHECK(Iso_neighbor_alltoall_init(NULL, 16, ISO_FLOAT, NULL, 64, ISO_BYTE, comm, &req) == ISO_SUCCESS);
    CHECK(Iso_request_get_stats(req, &st) == ISO_SUCCESS);
    CHECK(st.s == 7 && st.P == 120 && st.d == 3);
    CHECK(st.rounds == 3);                 /* one distinct non-zero coordinate per dimension */
    CHECK(st.parts == 3 * 1 + 3 * 2 + 3);  /* hops: three blocks with 1, three with 2, one with 3 */
    CHECK(st.bytes_min == 2LL * 120 * 7 * 64);
    CHECK(st.bytes_moved == 2LL * 120 * 12 * 64);
    CHECK(Iso_request_get_parts(req, parts, 64, &count) == ISO_SUCCESS);
    CHECK(count == 12);
    for (i = 0; i < count; i++) CHECK(parts[i].len == 64 && parts[i].dst_buf != ISO_BUF_SEND);
    CHECK(Iso_Start(req, NULL) == ISO_ERR_STATE); /* no buffers bound */
    CHECK(Iso_request_set_algorithm(req, ISO_ALG_DIRECT, 1) == ISO_SUCCESS);
    CHECK(Iso_request_get_stats(req, &st) == ISO_SUCCESS && st.rounds == 7 && st.bytes_moved == st.bytes_min);
    CHECK(Iso_request_set_algorithm(req, 99, 1) == ISO_ERR_ARG);
    CHECK(Iso_comm_free(&comm) == ISO_SUCCESS && comm == NULL);
    CHECK(Iso_request_free(&req) == ISO_SUCCESS && req == NULL);
    CHECK(Iso_neighborhood_create(0, dims, 7, octant, &comm) == ISO_ERR_DIMS && comm == NULL);
    CHECK(strlen(Iso_error_string(ISO_ERR_OVERLAP)) > 0);
    printf("c abi ok\n");
    return 0;
}
