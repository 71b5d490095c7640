/* A plain C program that runs a collective on the device through include/iso.h alone: the
 * worked example of Section II of the paper (Moore neighbourhood of radius 1 on a 4x4 torus,
 * block i of process q holds the single value 100*q + i) with buffers from cudaMalloc.
 * The expected rows are the hand-worked ones of tests/golden/moore_4x4_alltoall.txt. */
#include <stdio.h>
#include <string.h>

#include <cuda_runtime_api.h>

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
    int dims[2] = {4, 4};
    int moore[16] = {-1, -1, -1, 0, -1, 1, 0, -1, 0, 1, 1, -1, 1, 0, 1, 1};
    static const int want0[8] = {500, 401, 702, 103, 304, 1305, 1206, 1507};
    static const int want5[8] = {1000, 901, 802, 603, 404, 205, 106, 7};
    static const int want15[8] = {0, 301, 202, 1203, 1404, 805, 1106, 1007};
    int send[16 * 8], recv[16 * 8];
    int *d_send = NULL, *d_recv = NULL;
    Iso_comm comm = NULL;
    Iso_request req = NULL;
    int alg, q, i;

    for (q = 0; q < 16; q++)
        for (i = 0; i < 8; i++) send[q * 8 + i] = 100 * q + i;
    CHECK(cudaMalloc((void **)&d_send, sizeof send) == cudaSuccess);
    CHECK(cudaMalloc((void **)&d_recv, sizeof recv) == cudaSuccess);
    CHECK(cudaMemcpy(d_send, send, sizeof send, cudaMemcpyHostToDevice) == cudaSuccess);
    CHECK(Iso_neighborhood_create(2, dims, 8, moore, &comm) == ISO_SUCCESS);
    CHECK(Iso_neighbor_alltoall_init(d_send, 1, ISO_INT32, d_recv, 1, ISO_INT32, comm, &req) == ISO_SUCCESS);
    for (alg = ISO_ALG_COMBINING; alg <= ISO_ALG_TORUS; alg++) {
        CHECK(Iso_request_set_algorithm(req, alg, 1) == ISO_SUCCESS);
        CHECK(cudaMemset(d_recv, 0xA5, sizeof recv) == cudaSuccess);
        CHECK(Iso_Start(req, NULL) == ISO_SUCCESS);
        CHECK(Iso_wait(req) == ISO_SUCCESS);
        CHECK(cudaMemcpy(recv, d_recv, sizeof recv, cudaMemcpyDeviceToHost) == cudaSuccess);
        CHECK(memcmp(recv + 0 * 8, want0, sizeof want0) == 0);
        CHECK(memcmp(recv + 5 * 8, want5, sizeof want5) == 0);
        CHECK(memcmp(recv + 15 * 8, want15, sizeof want15) == 0);
    }
    CHECK(Iso_request_free(&req) == ISO_SUCCESS);
    CHECK(Iso_comm_free(&comm) == ISO_SUCCESS);
    cudaFree(d_send);
    cudaFree(d_recv);
    printf("c abi gpu ok\n");
    return 0;
}
