/* A kernel written by a USER of the library, compiled on its own against the public device
 * header: every PE (one work-group each, co-resident) puts its buffer to the next PE with the
 * work-group call, joins the in-kernel barrier, bumps a counter on PE 0 with a remote atomic,
 * scatters every other element to the previous PE with the strided call and finally takes part
 * in a device-resident sum reduction.  Only ishmemx_ctx(0) comes from the host library. */
#include <cuda_runtime.h>

#include "ishmem_device.cuh"

__global__ void __launch_bounds__(256) user_ring_step(const ishmem_ctx_t *ctxs, char *dst0, const char *src0,
                                                      size_t nbytes, long long *counter0, int *red_dst0,
                                                      const int *red_src0, size_t nred, int *status)
{
    const ishmem_ctx_t *ctx = ctxs + blockIdx.x;
    const long long off = ctx->heap_base - ctxs[0].heap_base; /* symmetric address -> my copy */
    char *dst = dst0 + off;
    const char *src = src0 + off;
    const int me = ishmem_my_pe(ctx), np = ishmem_n_pes(ctx);
    int rc = ishmemx_putmem_work_group(ctx, dst, src, nbytes, (me + 1) % np);
    rc |= ishmemx_barrier_all_work_group(ctx);
    if (threadIdx.x == 0)
        (void)ishmem_atomic_fetch_add<long long>(ctx, (long long *)((char *)counter0 + off), (long long)(me + 1), 0);
    /* every other 4-byte element of what I received goes to the second half of the previous PE's dst */
    ishmemx_iput_work_group<unsigned>(ctx, (unsigned *)(dst + nbytes), (const unsigned *)dst, 1, 2, nbytes / 8,
                                      (me + np - 1) % np);
    rc |= ishmemx_reduce_work_group<int, ISHMEM_OP_SUM>(ctx, ISHMEM_TEAM_WORLD, (int *)((char *)red_dst0 + off),
                                                        (const int *)((const char *)red_src0 + off), nred);
    if (rc && threadIdx.x == 0) atomicExch(status, rc);
}

extern "C" int user_launch_ring_step(const void *ctx0, int npes, void *dst, const void *src, size_t nbytes,
                                     void *counter, void *red_dst, const void *red_src, size_t nred, void *stream)
{
    int *d_status = nullptr;
    if (cudaMalloc((void **)&d_status, sizeof(int)) != cudaSuccess) return -100;
    cudaMemset(d_status, 0, sizeof(int));
    const ishmem_ctx_t *ctxs = (const ishmem_ctx_t *)ctx0;
    char *d = (char *)dst;
    const char *s = (const char *)src;
    long long *c = (long long *)counter;
    int *rd = (int *)red_dst;
    const int *rs = (const int *)red_src;
    void *params[] = {(void *)&ctxs, (void *)&d, (void *)&s, (void *)&nbytes, (void *)&c, (void *)&rd, (void *)&rs,
                      (void *)&nred, (void *)&d_status};
    /* the blocks wait on one another in the barrier: they must be co-resident */
    cudaError_t e = cudaLaunchCooperativeKernel((void *)user_ring_step, dim3(npes), dim3(256), params, 0,
                                                (cudaStream_t)stream);
    int status = -101;
    if (e == cudaSuccess && cudaStreamSynchronize((cudaStream_t)stream) == cudaSuccess)
        cudaMemcpy(&status, d_status, sizeof(int), cudaMemcpyDeviceToHost);
    cudaFree(d_status);
    return status;
}
