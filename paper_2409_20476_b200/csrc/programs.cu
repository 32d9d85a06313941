/* Device-initiated programs built on the device API: the put_signal / wait_until ping-pong
 * and the Jacobi overlap workload.  Both are co-resident (cooperative) launches in which
 * blocks of different PEs wait on one another with bounded waits. */
#include <algorithm>
#include <type_traits>
#include <vector>

#include "internal.h"

__device__ __forceinline__ char *local_of(const ishmem_ctx_t *ctxs, const ishmem_ctx_t *ctx, const void *sym0)
{
    return (char *)sym0 + (ctx->heap_base - ctxs[0].heap_base);
}

/* ---- ping-pong ------------------------------------------------------------------------- */

struct pingpong_out {
    unsigned long long elapsed_ns;
    unsigned long long mismatches;
};

__global__ void __launch_bounds__(1024) k_pingpong(const ishmem_ctx_t *ctxs, int pe_a, int pe_b, char *data0,
                                                   unsigned long long *sig0, size_t nbytes, int rounds,
                                                   pingpong_out *out)
{
    const bool is_a = (blockIdx.x == 0);
    /* the context in shared memory: each round translates two addresses right after an acquire */
    __shared__ ishmem_ctx_t ctx_copy;
    const ishmem_ctx_t *ctx = ctxs + (is_a ? pe_a : pe_b);
    const int other = is_a ? pe_b : pe_a;
    char *data = local_of(ctxs, ctx, data0);
    unsigned long long *sig = (unsigned long long *)local_of(ctxs, ctx, sig0);
    /* round stamps in the first and last 8 bytes of the payload catch a signal that
     * overtakes its data */
    volatile unsigned long long *w0 = (nbytes >= 8) ? (volatile unsigned long long *)data : nullptr;
    volatile unsigned long long *w1 =
        (nbytes >= 16 && nbytes % 8 == 0) ? (volatile unsigned long long *)(data + nbytes - 8) : nullptr;
    unsigned long long bad = 0, t0 = 0;
    ctx = ishmemx_ctx_stage_work_group(&ctx_copy, ctx);
    if (is_a && threadIdx.x == 0) t0 = ishmemi::globaltimer_ns();
    for (int r = 1; r <= rounds; ++r) {
        if (is_a) {
            if (threadIdx.x == 0) {
                if (w0) *w0 = (unsigned long long)r;
                if (w1) *w1 = (unsigned long long)r;
            }
            __syncthreads();
            ishmemx_putmem_signal_work_group(ctx, data, data, nbytes, sig, (unsigned long long)r,
                                             ISHMEM_SIGNAL_SET, other);
            if (ishmemx_uint64_wait_until_work_group(ctx, sig, ISHMEM_CMP_GE, (unsigned long long)r)) break;
        } else {
            if (ishmemx_uint64_wait_until_work_group(ctx, sig, ISHMEM_CMP_GE, (unsigned long long)r)) break;
            /* the leader checks the stamps while the others already start on the reply (both only
             * read this buffer; the leader signals last, after the barrier inside the put) */
            if (threadIdx.x == 0) {
                if (w0 && *w0 != (unsigned long long)r) ++bad;
                if (w1 && *w1 != (unsigned long long)r) ++bad;
            }
            ishmemx_putmem_signal_work_group(ctx, data, data, nbytes, sig, (unsigned long long)r,
                                             ISHMEM_SIGNAL_SET, other);
        }
    }
    if (threadIdx.x == 0) {
        if (is_a) out->elapsed_ns = ishmemi::globaltimer_ns() - t0;
        if (bad) atomicAdd(&out->mismatches, bad);
    }
}

extern "C" int ishmemx_pingpong(int pe_a, int pe_b, void *data, uint64_t *sig, size_t nbytes, int rounds,
                                int threads, double *half_rtt_ns, uint64_t *mismatches)
{
    ISHMEMI_REQUIRE_INIT();
    auto &g = g_ishmem;
    if (ishmemi_check_pe(pe_a) || ishmemi_check_pe(pe_b) || pe_a == pe_b) return ISHMEM_ERR_INVALID_PE;
    if (rounds < 1 || threads < 32 || threads > 1024) return ISHMEM_ERR_ARG;
    if ((uintptr_t)sig % 8 || (uintptr_t)data % 8) return ISHMEM_ERR_ALIGN;
    if (ishmemi_sym_offset(data, nbytes) < 0 || ishmemi_sym_offset(sig, 8) < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    cudaStream_t s;
    int rc = ishmemi_team_stream_begin(ISHMEM_TEAM_WORLD, &s);
    if (rc) return rc;
    pingpong_out *out = (pingpong_out *)g.h_pinned;
    out->elapsed_ns = 0;
    out->mismatches = 0;
    const ishmem_ctx_t *ctxs = g.d_ctx;
    char *d0 = (char *)data;
    unsigned long long *s0 = (unsigned long long *)sig;
    void *params[] = {(void *)&ctxs, (void *)&pe_a, (void *)&pe_b, (void *)&d0, (void *)&s0,
                      (void *)&nbytes, (void *)&rounds, (void *)&out};
    rc = ishmemi_cuda(cudaLaunchCooperativeKernel((void *)k_pingpong, dim3(2), dim3(threads), params, 0, s),
                      "cudaLaunchCooperativeKernel(pingpong)");
    ishmemi_count_launch();
    ishmemi_team_stream_end();
    if (rc) return rc;
    ISHMEMI_CUDA(cudaStreamSynchronize(s));
    if (half_rtt_ns) *half_rtt_ns = (double)out->elapsed_ns / (2.0 * rounds);
    if (mismatches) *mismatches = out->mismatches;
    return ISHMEM_OK;
}

/* ---- where a half round trip goes ------------------------------------------------------------
 * The same exchange as k_pingpong with the put_signal written out phase by phase (address translation,
 * copy, block barrier, release of the signal word, wait for the answer) and the SM's cycle counter
 * read between the phases by thread 0 of each block.  A thread issues in order, so a phase's count
 * includes the wait for whatever earlier load its first instruction needs: the counts say where the time
 * goes, not what each instruction costs in isolation.  staged: the context is read from a copy in
 * shared memory instead of from global memory.  The first block also times three primitives on its own
 * signal word: a dependent chain of relaxed loads (one trip to L2 each), a store followed by
 * st.release.gpu, and st.release.gpu with nothing pending. */
struct pingpong_phases {
    unsigned long long cycles[2][5]; /* per block: wait / translate / copy / barrier / release */
    unsigned long long prim[3];      /* L2 trip, store + release, release alone: cycles per operation */
    unsigned long long elapsed_ns;
};

__global__ void __launch_bounds__(1024) k_pingpong_phases(const ishmem_ctx_t *ctxs, int pe_a, int pe_b, char *data0,
                                                          unsigned long long *sig0, size_t nbytes, int rounds, int staged,
                                                          pingpong_phases *out)
{
    const bool is_a = (blockIdx.x == 0);
    __shared__ ishmem_ctx_t ctx_copy;
    const ishmem_ctx_t *ctx = ctxs + (is_a ? pe_a : pe_b);
    const int other = is_a ? pe_b : pe_a;
    char *data = local_of(ctxs, ctx, data0);
    unsigned long long *sig = (unsigned long long *)local_of(ctxs, ctx, sig0);
    if (staged) ctx = ishmemx_ctx_stage_work_group(&ctx_copy, ctx);
    unsigned long long acc[5] = {0, 0, 0, 0, 0}, t_start = 0;
    const unsigned tid = threadIdx.x;
    if (is_a && tid == 0) t_start = ishmemi::globaltimer_ns();
    __shared__ int give_up;
    if (tid == 0) give_up = 0;
    __syncthreads();
    for (int r = 1; r <= rounds; ++r) {
        long long c0 = clock64();
        if (!is_a) { /* B answers: it waits first */
            if (tid == 0 && ishmem_uint64_wait_until(ctx, sig, ISHMEM_CMP_GE, (unsigned long long)r)) give_up = 1;
            __syncthreads();
            if (give_up) break;
        }
        long long c1 = clock64();
        char *rdst = ishmemi::translate(ctx, data, other);
        unsigned long long *rs = ishmemi::translate(ctx, sig, other);
        if (!rdst || !rs) break;
        /* consume the translated addresses so that the wait for the context reads is counted here */
        asm volatile("" ::"l"(rdst), "l"(rs) : "memory");
        long long c2 = clock64();
        ishmemi::copy_bytes(rdst, data, nbytes, tid, blockDim.x);
        long long c3 = clock64();
        __syncthreads();
        long long c4 = clock64();
        if (tid == 0) ishmemi::st_release(rs, (unsigned long long)r);
        long long c5 = clock64();
        if (is_a) {
            if (tid == 0 && ishmem_uint64_wait_until(ctx, sig, ISHMEM_CMP_GE, (unsigned long long)r)) give_up = 1;
            __syncthreads();
            if (give_up) break;
        }
        long long c6 = clock64();
        acc[0] += (unsigned long long)((c1 - c0) + (c6 - c5));
        acc[1] += (unsigned long long)(c2 - c1);
        acc[2] += (unsigned long long)(c3 - c2);
        acc[3] += (unsigned long long)(c4 - c3);
        acc[4] += (unsigned long long)(c5 - c4);
    }
    if (tid == 0) {
        for (int i = 0; i < 5; ++i) out->cycles[blockIdx.x][i] = acc[i];
        if (is_a) {
            out->elapsed_ns = ishmemi::globaltimer_ns() - t_start;
            /* primitives, on a word of this PE's own signal area that nobody else touches */
            unsigned long long *w = sig + 2;
            const int n = 256;
            unsigned long long v = 0;
            long long p0 = clock64();
            for (int i = 0; i < n; ++i) v += ishmemi::ld_relaxed(w + (v & 1));
            long long p1 = clock64();
            for (int i = 0; i < n; ++i) {
                *(volatile unsigned long long *)(w + 1) = v + (unsigned long long)i;
                ishmemi::st_release(w, 0ull);
            }
            long long p2 = clock64();
            for (int i = 0; i < n; ++i) ishmemi::st_release(w, 0ull);
            long long p3 = clock64();
            out->prim[0] = (unsigned long long)(p1 - p0) / n;
            out->prim[1] = (unsigned long long)(p2 - p1) / n;
            out->prim[2] = (unsigned long long)(p3 - p2) / n;
            *(volatile unsigned long long *)(w + 1) = 0;
        }
    }
}

extern "C" int ishmemx_pingpong_phases(int pe_a, int pe_b, void *data, uint64_t *sig, size_t nbytes, int rounds,
                                       int threads, int staged, double *ns_out)
{
    ISHMEMI_REQUIRE_INIT();
    auto &g = g_ishmem;
    if (ishmemi_check_pe(pe_a) || ishmemi_check_pe(pe_b) || pe_a == pe_b) return ISHMEM_ERR_INVALID_PE;
    if (rounds < 1 || threads < 32 || threads > 1024 || !ns_out) return ISHMEM_ERR_ARG;
    if ((uintptr_t)sig % 8 || (uintptr_t)data % 8) return ISHMEM_ERR_ALIGN;
    if (ishmemi_sym_offset(data, nbytes) < 0 || ishmemi_sym_offset(sig, 32) < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    cudaStream_t s;
    int rc = ishmemi_team_stream_begin(ISHMEM_TEAM_WORLD, &s);
    if (rc) return rc;
    pingpong_phases *out = (pingpong_phases *)g.h_pinned;
    memset(out, 0, sizeof(*out));
    const ishmem_ctx_t *ctxs = g.d_ctx;
    char *d0 = (char *)data;
    unsigned long long *s0 = (unsigned long long *)sig;
    void *params[] = {(void *)&ctxs, (void *)&pe_a,  (void *)&pe_b,   (void *)&d0, (void *)&s0,
                      (void *)&nbytes, (void *)&rounds, (void *)&staged, (void *)&out};
    rc = ishmemi_cuda(cudaLaunchCooperativeKernel((void *)k_pingpong_phases, dim3(2), dim3(threads), params, 0, s),
                      "cudaLaunchCooperativeKernel(pingpong_phases)");
    ishmemi_count_launch();
    ishmemi_team_stream_end();
    if (rc) return rc;
    ISHMEMI_CUDA(cudaStreamSynchronize(s));
    int khz = 0;
    ISHMEMI_CUDA(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, g.device));
    const double ns_per_cycle = 1e6 / (double)khz;
    for (int b = 0; b < 2; ++b)
        for (int i = 0; i < 5; ++i) ns_out[b * 5 + i] = (double)out->cycles[b][i] * ns_per_cycle / rounds;
    for (int i = 0; i < 3; ++i) ns_out[10 + i] = (double)out->prim[i] * ns_per_cycle;
    ns_out[13] = (double)out->elapsed_ns / (2.0 * rounds);
    return ISHMEM_OK;
}

/* ---- device-timed put/get latency --------------------------------------------------------- */

template <int LEVEL>
__global__ void __launch_bounds__(1024) k_rma_latency(const ishmem_ctx_t *ctxs, int my_pe, char *dest,
                                                      const char *src, size_t nbytes, int pe, int is_get,
                                                      int iters, unsigned staging_bytes, unsigned long long *elapsed_ns)
{
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ ishmem_ctx_t ctx_copy;
    const ishmem_ctx_t *ctx = ishmemx_ctx_stage_work_group(&ctx_copy, ctxs + my_pe);
    ishmemx_staging_t st = {nullptr, 0};
    if (LEVEL == ISHMEMX_WORK_GROUP_BULK) {
        st.smem = dyn_smem;
        st.bytes = staging_bytes;
    }
    __syncthreads();
    unsigned long long t0 = 0;
    if (threadIdx.x == 0) t0 = ishmemi::globaltimer_ns();
    for (int it = 0; it < iters; ++it) {
        if (LEVEL == ISHMEMX_WORK_ITEM) {
            if (threadIdx.x == 0) {
                if (is_get) ishmem_getmem(ctx, dest, src, nbytes, pe);
                else ishmem_putmem(ctx, dest, src, nbytes, pe);
                ishmem_quiet(ctx);
            }
        } else if (LEVEL == ISHMEMX_SUB_GROUP) {
            if (threadIdx.x < 32u) {
                if (is_get) ishmemx_getmem_sub_group(ctx, dest, src, nbytes, pe);
                else ishmemx_putmem_sub_group(ctx, dest, src, nbytes, pe);
                ishmem_quiet(ctx);
            }
        } else if (LEVEL == ISHMEMX_WORK_GROUP_ENGINE) {
            int rc = is_get ? ishmemx_getmem_engine_work_group(ctx, dest, src, nbytes, pe)
                            : ishmemx_putmem_engine_work_group(ctx, dest, src, nbytes, pe);
            if (rc) break;
        } else {
            int rc = is_get ? ishmemx_getmem_work_group(ctx, dest, src, nbytes, pe, st)
                            : ishmemx_putmem_work_group(ctx, dest, src, nbytes, pe, st);
            ishmemx_quiet_work_group(ctx);
            if (rc) break; /* latched; same value in every thread */
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) *elapsed_ns = ishmemi::globaltimer_ns() - t0;
}

extern "C" int ishmemx_rma_latency(int my_pe, void *dest, const void *src, size_t nbytes, int pe, int is_get,
                                   int level, int threads, int iters, double *ns_per_op)
{
    ISHMEMI_REQUIRE_INIT();
    auto &g = g_ishmem;
    if (ishmemi_check_pe(my_pe) || ishmemi_check_pe(pe)) return ISHMEM_ERR_INVALID_PE;
    if (iters < 1 || threads < 1 || threads > 1024 || !ns_per_op) return ISHMEM_ERR_ARG;
    if (level < ISHMEMX_WORK_ITEM || level > ISHMEMX_WORK_GROUP_ENGINE) return ISHMEM_ERR_ARG;
    if (level == ISHMEMX_SUB_GROUP && threads < 32) return ISHMEM_ERR_ARG;
    if (level == ISHMEMX_WORK_GROUP_ENGINE && g.h_ctx[0].proxy == nullptr) return ISHMEM_ERR_ARG;
    if (nbytes && (!dest || !src)) return ISHMEM_ERR_ARG;
    if (ishmemi_sym_offset(is_get ? src : (const void *)dest, nbytes) < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    char *dl = ishmemi_localise(dest, nbytes, my_pe);
    const char *sl = ishmemi_localise(src, nbytes, my_pe);
    unsigned long long *out = (unsigned long long *)g.h_pinned;
    *out = 0;
    unsigned staging = 0;
    cudaStream_t s = ishmemi_pe_stream_for_op(my_pe);
    const ishmem_ctx_t *ctxs = g.d_ctx;
    switch (level) {
    case ISHMEMX_WORK_ITEM:
        k_rma_latency<ISHMEMX_WORK_ITEM><<<1, threads, 0, s>>>(ctxs, my_pe, dl, sl, nbytes, pe, is_get, iters, 0, out);
        break;
    case ISHMEMX_SUB_GROUP:
        k_rma_latency<ISHMEMX_SUB_GROUP><<<1, threads, 0, s>>>(ctxs, my_pe, dl, sl, nbytes, pe, is_get, iters, 0, out);
        break;
    case ISHMEMX_WORK_GROUP:
        k_rma_latency<ISHMEMX_WORK_GROUP><<<1, threads, 0, s>>>(ctxs, my_pe, dl, sl, nbytes, pe, is_get, iters, 0, out);
        break;
    case ISHMEMX_WORK_GROUP_ENGINE:
        k_rma_latency<ISHMEMX_WORK_GROUP_ENGINE><<<1, threads, 0, s>>>(ctxs, my_pe, dl, sl, nbytes, pe, is_get, iters, 0,
                                                                        out);
        break;
    default: {
        static unsigned smem = 0;
        if (!smem) {
            unsigned want = 192 * 1024 + 128;
            if (want > g.max_dyn_smem) want = (unsigned)g.max_dyn_smem;
            ISHMEMI_CUDA(cudaFuncSetAttribute(k_rma_latency<ISHMEMX_WORK_GROUP_BULK>,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize, (int)want));
            smem = want;
        }
        staging = smem;
        k_rma_latency<ISHMEMX_WORK_GROUP_BULK><<<1, threads, staging, s>>>(ctxs, my_pe, dl, sl, nbytes, pe, is_get,
                                                                          iters, staging, out);
    }
    }
    ishmemi_count_launch();
    int rc = ishmemi_check_launch("k_rma_latency");
    if (rc) return rc;
    ISHMEMI_CUDA(cudaStreamSynchronize(s));
    *ns_per_op = (double)*out / (double)iters;
    return ISHMEM_OK;
}

/* ---- cutover tuning from measurement (Section 4) ----------------------------------------------- */

/* mean time in ns of one host-initiated ishmem_putmem PE 0 -> PE `to` under the current cutover */
static int time_host_put(void *dst, const void *src, size_t n, int to, int reps, double *ns)
{
    auto &g = g_ishmem;
    cudaEvent_t a, b;
    ISHMEMI_CUDA(cudaEventCreate(&a));
    ISHMEMI_CUDA(cudaEventCreate(&b));
    int rc = ishmem_putmem(0, dst, src, n, to); /* warm-up; also joins pending team work */
    cudaStream_t s = g.pe_stream[0];
    if (!rc) rc = ishmemi_cuda(cudaEventRecord(a, s), "cudaEventRecord");
    for (int i = 0; i < reps && !rc; ++i) rc = ishmem_putmem(0, dst, src, n, to);
    if (!rc) rc = ishmemi_cuda(cudaEventRecord(b, s), "cudaEventRecord");
    if (!rc) rc = ishmemi_cuda(cudaEventSynchronize(b), "cudaEventSynchronize");
    float ms = 0.f;
    if (!rc) rc = ishmemi_cuda(cudaEventElapsedTime(&ms, a, b), "cudaEventElapsedTime");
    cudaEventDestroy(a);
    cudaEventDestroy(b);
    *ns = (double)ms * 1e6 / reps;
    return rc;
}

extern "C" int ishmemx_tune_cutover(int which, int threads, size_t max_bytes, size_t *chosen)
{
    ISHMEMI_REQUIRE_INIT();
    auto &g = g_ishmem;
    if (which != 0 && which != 3) return ISHMEM_ERR_ARG;
    if (which == 3 && (g.h_ctx[0].proxy == nullptr || threads < 1 || threads > 1024)) return ISHMEM_ERR_ARG;
    if (max_bytes < 4096) return ISHMEM_ERR_ARG;
    void *src = ishmem_malloc(max_bytes), *dst = ishmem_malloc(max_bytes);
    if (!src || !dst) {
        ishmem_free(src);
        ishmem_free(dst);
        return ISHMEM_ERR_OOM;
    }
    const int to = g.npes > 1 ? 1 : 0;
    const size_t saved = ishmemx_get_cutover(which), saved_upto = ishmemx_get_cutover(5);
    int rc = 0;
    /* The engine "wins" a size when it is at least as fast there.
     * which = 3: sizes 4 KiB, 16 KiB, ...; the cutover is the start of the unbroken run of wins at
     * the top.
     * which = 0: sizes 4 KiB, 8 KiB, ...; the engine gets the LONGEST run of consecutive wins,
     * [pick, upto): on this GPU it wins a middle range and loses or ties above it, which one
     * threshold cannot say. */
    size_t pick = (size_t)-1, upto = (size_t)-1;
    size_t run_lo = (size_t)-1, best_lo = (size_t)-1, best_hi = (size_t)-1;
    int run_len = 0, best_len = 0;
    if (which == 0) ishmemx_set_cutover(5, (size_t)-1);
    for (size_t n = 4096; n <= max_bytes && !rc; n *= (which == 0 ? 2 : 4)) {
        double t_ldst = 0, t_engine = 0;
        const int reps = n <= (1u << 20) ? 50 : (n <= (16u << 20) ? 10 : 3);
        if (which == 0) {
            ishmemx_set_cutover(0, (size_t)-1);
            rc = time_host_put(dst, src, n, to, reps, &t_ldst);
            ishmemx_set_cutover(0, 0);
            if (!rc) rc = time_host_put(dst, src, n, to, reps, &t_engine);
        } else {
            ishmemx_set_cutover(3, (size_t)-1);
            rc = ishmemx_rma_latency(0, dst, src, n, to, 0, ISHMEMX_WORK_GROUP, threads, reps, &t_ldst);
            if (!rc) rc = ishmemx_rma_latency(0, dst, src, n, to, 0, ISHMEMX_WORK_GROUP_ENGINE, threads, reps, &t_engine);
        }
        if (t_engine <= t_ldst) {
            if (pick == (size_t)-1) pick = n;
            if (run_len++ == 0) run_lo = n;
            if (run_len > best_len) best_len = run_len, best_lo = run_lo, best_hi = (size_t)-1;
        } else {
            pick = (size_t)-1;
            if (run_len && run_len == best_len && best_hi == (size_t)-1) best_hi = n; /* first loss after the best run */
            run_len = 0;
        }
    }
    if (which == 0) {
        pick = best_lo;
        upto = best_hi;
        ishmemx_set_cutover(5, rc ? saved_upto : upto);
    }
    ishmemx_set_cutover(which, rc ? saved : pick);
    cudaDeviceSynchronize();
    ishmem_free(src);
    ishmem_free(dst);
    if (!rc && chosen) *chosen = pick;
    return rc;
}

/* ---- Jacobi overlap workload -------------------------------------------------------------- */

struct jacobi_args {
    double *buf0, *buf1;          /* PE 0's copies */
    unsigned long long *sig;      /* [0]: halo from the PE above arrived, [1]: from below */
    size_t ny, nx;
    int iters, overlap, groups;
    unsigned long long *done;     /* scratch [npes*groups]: sweeps completed by each block */
    double *partial;              /* scratch [npes*groups]: residual partial sums */
    int sliding;                  /* even nx: interior rows by the register sliding window */
    int colsplit;                 /* the blocks of a PE split the strip by columns (else by rows) */
};

__device__ __forceinline__ void strip_of(size_t ny, int npes, int pe, size_t *first, size_t *rows)
{
    const size_t base = ny / (size_t)npes, extra = ny % (size_t)npes;
    *rows = base + ((size_t)pe < extra ? 1 : 0);
    *first = (size_t)pe * base + ((size_t)pe < extra ? (size_t)pe : extra);
}

/* One local row r of the strip: nxt[r] = sweep(cur[r-1..r+1]); boundary cells are copied.
 * Adds the squared update to *acc when want_res. */
__device__ __forceinline__ void jacobi_row(const double *cur, double *nxt, size_t r, size_t nx, bool fixed_row,
                                           unsigned tid, unsigned nthr, bool want_res, double *acc, size_t c_lo = 0,
                                           size_t c_hi = ~(size_t)0)
{
    const double *up = cur + (r - 1) * nx, *mid = cur + r * nx, *dn = cur + (r + 1) * nx;
    double *out = nxt + r * nx;
    if (c_hi > nx) c_hi = nx;
    if (fixed_row) {
        for (size_t j = c_lo + tid; j < c_hi; j += nthr) out[j] = mid[j];
        return;
    }
    if ((nx & 1) == 0 && c_lo == 0 && c_hi == nx) {
        const size_t half = nx >> 1;
        for (size_t c = tid; c < half; c += nthr) {
            const size_t j = c << 1;
            const double2 u = *(const double2 *)(up + j);
            const double2 d = *(const double2 *)(dn + j);
            const double2 m = *(const double2 *)(mid + j);
            const double left = (j > 0) ? mid[j - 1] : 0.0;
            const double right = (j + 2 < nx) ? mid[j + 2] : 0.0;
            double2 v;
            v.x = (j == 0) ? m.x : 0.25 * ((u.x + d.x) + (left + m.y));
            v.y = (j + 2 == nx) ? m.y : 0.25 * ((u.y + d.y) + (m.x + right));
            *(double2 *)(out + j) = v;
            if (want_res) {
                const double dx = v.x - m.x, dy = v.y - m.y;
                *acc += dx * dx;
                *acc += dy * dy;
            }
        }
        return;
    }
    for (size_t j = c_lo + tid; j < c_hi; j += nthr) {
        double v = mid[j];
        if (j > 0 && j + 1 < nx) v = 0.25 * ((up[j] + dn[j]) + (mid[j - 1] + mid[j + 1]));
        out[j] = v;
        if (want_res) {
            const double dd = v - mid[j];
            *acc += dd * dd;
        }
    }
}


/* ---- register sliding window ------------------------------------------------------------------
 * Rows [ra, rb) of the strip (local row numbers) for even nx.  Each warp takes tiles of 60 output
 * columns: its 32 lanes load the 64 columns around them (one aligned double2 per lane, so the
 * tile's left and right neighbour columns are lanes 0 and 31) and walk down the rows.  The rows
 * above and at the current position stay in registers, DEPTH further rows are already on their
 * way (independent 16-byte loads, refilled one per step), and the left/right neighbours of a
 * lane's pair come from the adjacent lanes by shuffle; lanes 1..30 store.  Every element of `cur`
 * is loaded once per sweep (plus 4 of every 64 a second time, from cache), every element of `nxt`
 * stored once, and there is no block-wide barrier inside.  The arithmetic is the same expression,
 * in the same order, as jacobi_row.  fixed0 / fixed1: local numbers of the rows that are the
 * grid's first and last row (kept as they are), or ~0u when they lie outside this strip.
 * Returns this thread's share of the squared update when want_res. */
template <int DEPTH, bool FIXED = true, bool RES = true>
__device__ __forceinline__ double jacobi_march_tiles(const double *cur, double *nxt, unsigned ra, unsigned rb,
                                                     unsigned fixed0, unsigned fixed1, unsigned nx, bool want_res,
                                                     unsigned t_lo, unsigned t_hi)
{
    /* FIXED = false: the caller knows that none of the rows is the grid's first or last one;
     * RES = false: no residual wanted -- both spare the loop a few registers */
    double acc = 0.0;
    if (rb <= ra) return acc;
    const unsigned lane = threadIdx.x & 31u, nwarps = blockDim.x >> 5;
    const unsigned full = 0xffffffffu;
    const double2 zero = make_double2(0.0, 0.0);
    for (unsigned t = t_lo + (threadIdx.x >> 5); t < t_hi; t += nwarps) {
        const int jl = (int)(t * 60u) - 2 + 2 * (int)lane; /* first column of this lane's pair */
        const bool ld_ok = jl >= 0 && jl < (int)nx;
        const bool st_ok = ld_ok && lane >= 1 && lane <= 30;
        const unsigned j = ld_ok ? (unsigned)jl : 0u;
        const double *pl = cur + (size_t)(ra - 1) * nx + j; /* next row to load */
        double2 up = ld_ok ? *(const double2 *)pl : zero;
        pl += nx;
        double2 mid = ld_ok ? *(const double2 *)pl : zero;
        pl += nx;
        double2 f[DEPTH];
        unsigned loaded = ra + 1; /* local row number pl points at */
#pragma unroll
        for (int s = 0; s < DEPTH; ++s) {
            f[s] = zero;
            if (loaded <= rb) {
                if (ld_ok) f[s] = *(const double2 *)pl;
                pl += nx;
                ++loaded;
            }
        }
        double ml = __shfl_up_sync(full, mid.y, 1), mr = __shfl_down_sync(full, mid.x, 1);
        double *po = nxt + (size_t)ra * nx + j;
        for (unsigned r = ra; r < rb; r += DEPTH) {
#pragma unroll
            for (int s = 0; s < DEPTH; ++s) {
                if (r + s < rb) { /* uniform over the warp */
                    const double2 dn = f[s];
                    if (loaded <= rb) { /* refill this slot with the row DEPTH further down */
                        if (ld_ok) f[s] = *(const double2 *)pl;
                        pl += nx;
                        ++loaded;
                    }
                    double2 o = mid;
                    if (!FIXED || (r + s != fixed0 && r + s != fixed1)) {
                        if (j != 0) o.x = 0.25 * ((up.x + dn.x) + (ml + mid.y));
                        if (j + 2 != nx) o.y = 0.25 * ((up.y + dn.y) + (mid.x + mr));
                        if (RES && want_res && st_ok) {
                            const double dx = o.x - mid.x, dy = o.y - mid.y;
                            acc += dx * dx;
                            acc += dy * dy;
                        }
                    }
                    if (st_ok) *(double2 *)po = o;
                    po += nx;
                    up = mid;
                    mid = dn;
                    ml = __shfl_up_sync(full, dn.y, 1);
                    mr = __shfl_down_sync(full, dn.x, 1);
                }
            }
        }
    }
    return acc;
}

/* out of line, so that the window gets a register allocation of its own: all tiles of the rows
 * (two values fewer to carry), or the tiles [t_lo, t_hi) */
template <int DEPTH>
static __device__ __noinline__ double jacobi_march(const double *cur, double *nxt, unsigned ra, unsigned rb,
                                                   unsigned fixed0, unsigned fixed1, unsigned nx, bool want_res)
{
    return jacobi_march_tiles<DEPTH>(cur, nxt, ra, rb, fixed0, fixed1, nx, want_res, 0u, (nx + 59u) / 60u);
}
template <int DEPTH>
static __device__ __noinline__ double jacobi_march_range(const double *cur, double *nxt, unsigned ra, unsigned rb,
                                                         unsigned fixed0, unsigned fixed1, unsigned nx, bool want_res,
                                                         unsigned t_lo, unsigned t_hi)
{
    return jacobi_march_tiles<DEPTH>(cur, nxt, ra, rb, fixed0, fixed1, nx, want_res, t_lo, t_hi);
}

/* The first and the last row of a block's range (local rows rA and rB; rB == ~0u: only rA), which
 * are computed after the neighbours' rows have arrived.  Same 60-column tiles and shuffles as
 * jacobi_march; the loads of U tiles x 2 rows x 3 source rows are all issued before the first
 * use, since there is nothing to slide along. */
template <int U>
__device__ __forceinline__ double jacobi_edge_rows(const double *cur, double *nxt, unsigned rA, unsigned rB,
                                                   unsigned fixed0, unsigned fixed1, unsigned nx, bool want_res,
                                                   unsigned t_lo, unsigned ntiles)
{
    double acc = 0.0;
    const unsigned lane = threadIdx.x & 31u, nwarps = blockDim.x >> 5;
    const unsigned full = 0xffffffffu;
    const double2 zero = make_double2(0.0, 0.0);
    const unsigned rows[2] = {rA, rB};
    for (unsigned t0 = t_lo + (threadIdx.x >> 5) * U; t0 < ntiles; t0 += nwarps * U) {
        double2 up[U][2], mid[U][2], dn[U][2];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int jl = (int)((t0 + k) * 60u) - 2 + 2 * (int)lane;
            const bool ld_ok = t0 + k < ntiles && jl >= 0 && jl < (int)nx;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                up[k][e] = mid[k][e] = dn[k][e] = zero;
                if (ld_ok && rows[e] != ~0u) {
                    const double *pm = cur + (size_t)rows[e] * nx + jl;
                    up[k][e] = *(const double2 *)(pm - nx);
                    mid[k][e] = *(const double2 *)pm;
                    dn[k][e] = *(const double2 *)(pm + nx);
                }
            }
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const int jl = (int)((t0 + k) * 60u) - 2 + 2 * (int)lane;
            const bool st_ok = t0 + k < ntiles && jl >= 0 && jl < (int)nx && lane >= 1 && lane <= 30;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const double2 m = mid[k][e];
                const double ml = __shfl_up_sync(full, m.y, 1), mr = __shfl_down_sync(full, m.x, 1);
                if (!st_ok || rows[e] == ~0u) continue;
                double2 o = m;
                if (rows[e] != fixed0 && rows[e] != fixed1) {
                    if (jl != 0) o.x = 0.25 * ((up[k][e].x + dn[k][e].x) + (ml + m.y));
                    if (jl + 2 != (int)nx) o.y = 0.25 * ((up[k][e].y + dn[k][e].y) + (m.x + mr));
                    if (want_res) {
                        const double dx = o.x - m.x, dy = o.y - m.y;
                        acc += dx * dx;
                        acc += dy * dy;
                    }
                }
                *(double2 *)(nxt + (size_t)rows[e] * nx + jl) = o;
            }
        }
    }
    return acc;
}

/* MAXT: largest block the instance may be launched with (it fixes the registers per thread);
 * DEPTH: rows in flight per lane in the sliding window.
 *
 * The G blocks of a PE share its strip in one of two ways.
 *  - by rows (colsplit = 0): block g takes a band of rows and walks every column tile of it;
 *    it sends the strip's first / last row when it owns them, and before its band's two edge
 *    rows it waits for the blocks above and below (or the neighbour PE's halo).
 *  - by columns (colsplit = 1): block g takes a range of 60-column tiles and walks them down the
 *    whole strip, one warp per tile when the block is large enough, so that the warps of a PE
 *    advance together through one band of rows (a short contiguous window of memory, which this
 *    GPU serves faster than many scattered streams).  Every block sends its columns of the first
 *    and last row (the signal counts the pieces), and at the start of a sweep waits for the
 *    blocks left and right of it, whose columns its outermost tiles overlap by two. */
template <int MAXT, int DEPTH>
__global__ void __launch_bounds__(MAXT) k_jacobi(const ishmem_ctx_t *ctxs, jacobi_args a)
{
    const int P = ctxs[0].npes, G = a.groups;
    const int p = (int)blockIdx.x / G, g = (int)blockIdx.x % G;
    __shared__ ishmem_ctx_t ctx_copy; /* every sweep's put_signal and wait read the context after an acquire */
    const ishmem_ctx_t *ctx = ctxs + p;
    const unsigned tid = threadIdx.x, nthr = blockDim.x;
    size_t first, rows, rows_above = 0, f2;
    strip_of(a.ny, P, p, &first, &rows);
    if (p > 0) strip_of(a.ny, P, p - 1, &f2, &rows_above);
    double *b[2] = {(double *)local_of(ctxs, ctx, a.buf0), (double *)local_of(ctxs, ctx, a.buf1)};
    unsigned long long *sig = (unsigned long long *)local_of(ctxs, ctx, a.sig);
    const size_t nx = a.nx;
    const bool cols = a.colsplit != 0;
    /* this block's local rows [r0, r1) out of 1..rows, and its tiles [t_lo, t_hi) of 60 columns */
    const size_t r0 = cols ? 1 : 1 + rows * (size_t)g / (size_t)G;
    const size_t r1 = cols ? rows + 1 : 1 + rows * (size_t)(g + 1) / (size_t)G;
    const unsigned ntiles = (unsigned)((nx + 59) / 60);
    const unsigned t_lo = cols ? (unsigned)((size_t)ntiles * (size_t)g / (size_t)G) : 0u;
    const unsigned t_hi = cols ? (unsigned)((size_t)ntiles * (size_t)(g + 1) / (size_t)G) : ntiles;
    const size_t c_lo = (size_t)t_lo * 60, c_hi = ((size_t)t_hi * 60 < nx) ? (size_t)t_hi * 60 : nx;
    unsigned long long *done = a.done + (size_t)p * G;
    double acc = 0.0;
    __shared__ int give_up;
    /* even nx: register sliding window; odd nx: row by row with scalar accesses */
    const bool slide = a.sliding != 0;
    /* local numbers of the grid's first and last row when they belong to this strip */
    const unsigned fixed0 = (first == 0) ? 1u : ~0u;
    const unsigned fixed1 = (first + rows == a.ny) ? (unsigned)rows : ~0u;
    /* Halo signals.  By rows one block sends the whole row and SETs the word to the sweep number.
     * By columns every block sends its piece and ADDs 1, and the words alternate with the parity
     * of the sweep (sig[2], sig[3] for even sweeps): a PE can receive pieces of the next sweep
     * while it still waits for one of this sweep -- never of the sweep after that, which needs
     * this PE's own next halo -- so a word only ever counts sweeps up to the one waited for. */
    if (tid == 0) give_up = 0;
    ctx = ishmemx_ctx_stage_work_group(&ctx_copy, ctx); /* ends with the block barrier */

    /* rows [ra, rb) of this block's columns */
    auto sweep_rows = [&](const double *cur, double *nxt, size_t ra, size_t rb, bool want_res) {
        if (rb <= ra) return;
        if (slide) {
            acc += cols ? jacobi_march_range<DEPTH>(cur, nxt, (unsigned)ra, (unsigned)rb, fixed0, fixed1, (unsigned)nx,
                                                    want_res, t_lo, t_hi)
                        : jacobi_march<DEPTH>(cur, nxt, (unsigned)ra, (unsigned)rb, fixed0, fixed1, (unsigned)nx,
                                              want_res);
        } else {
            for (size_t r = ra; r < rb; ++r) {
                const size_t gi = first + r - 1;
                jacobi_row(cur, nxt, r, nx, gi == 0 || gi == a.ny - 1, tid, nthr, want_res, &acc, c_lo, c_hi);
            }
        }
    };
    /* the two rows rA and rB (rB == ~0: only rA) of this block's columns */
    auto two_rows = [&](const double *cur, double *nxt, size_t rA, size_t rB, bool want_res) {
        if (slide) {
            acc += jacobi_edge_rows<(MAXT <= 512) ? 2 : 1>(cur, nxt, (unsigned)rA, rB == ~(size_t)0 ? ~0u : (unsigned)rB,
                                                           fixed0, fixed1, (unsigned)nx, want_res, t_lo, t_hi);
        } else {
            sweep_rows(cur, nxt, rA, rA + 1, want_res);
            if (rB != ~(size_t)0) sweep_rows(cur, nxt, rB, rB + 1, want_res);
        }
    };
    /* block `other` of this PE has finished sweep it - 1 */
    auto wait_block = [&](int other, int it, ishmemi::deadline &dl) -> int {
        while (ishmemi::ld_acquire(done + other) < (unsigned long long)it)
            if (dl.expired()) return ISHMEM_ERR_TIMEOUT;
        return 0;
    };

    for (int it = 0; it < a.iters; ++it) {
        const double *cur = b[it & 1];
        double *nxt = b[(it + 1) & 1];
        const unsigned long long round = (unsigned long long)it + 1;
        const bool want_res = (it == a.iters - 1);
        if (cols && G > 1) {
            /* the blocks left and right have finished the previous sweep: their columns next to
             * mine are current, and they no longer read the columns I am about to overwrite */
            if (tid == 0) {
                ishmemi::deadline dl(ctx->wait_limit_ns);
                int rc = (g > 0) ? wait_block(g - 1, it, dl) : 0;
                if (!rc && g < G - 1) rc = wait_block(g + 1, it, dl);
                if (rc) {
                    ishmemi::latch_error(ctx, rc);
                    give_up = 1;
                }
            }
            __syncthreads();
            if (give_up) break;
        }
        /* (a) halo rows of the current sweep go out first: my first row to the bottom halo of
         * the PE above, my last row to the top halo of the PE below */
        unsigned long long *sig_top = sig + 0, *sig_bottom = sig + 1; /* halo from above / below arrived */
        unsigned long long expect = round;
        if (cols) {
            sig_top += 2 * (it & 1);
            sig_bottom += 2 * (it & 1);
            expect = (unsigned long long)G * (unsigned long long)(it / 2 + 1);
            if (p > 0)
                ishmemx_putmem_signal_work_group(ctx, (void *)(cur + (rows_above + 1) * nx + c_lo), cur + nx + c_lo,
                                                 (c_hi - c_lo) * 8, sig_bottom, 1, ISHMEM_SIGNAL_ADD, p - 1);
            if (p + 1 < P)
                ishmemx_putmem_signal_work_group(ctx, (void *)(cur + c_lo), cur + rows * nx + c_lo, (c_hi - c_lo) * 8,
                                                 sig_top, 1, ISHMEM_SIGNAL_ADD, p + 1);
        } else {
            if (g == 0 && p > 0)
                ishmemx_putmem_signal_work_group(ctx, (void *)(cur + (rows_above + 1) * nx), cur + nx, nx * 8, sig + 1,
                                                 round, ISHMEM_SIGNAL_SET, p - 1);
            if (g == G - 1 && p + 1 < P)
                ishmemx_putmem_signal_work_group(ctx, (void *)cur, cur + rows * nx, nx * 8, sig + 0, round,
                                                 ISHMEM_SIGNAL_SET, p + 1);
        }
        /* (b) rows that need nobody else's data of this sweep */
        if (a.overlap && r1 > r0 + 2) sweep_rows(cur, nxt, r0 + 1, r1 - 1, want_res);
        /* (c) wait for the rows above and below this block's range: neighbouring blocks of
         * the same PE publish a sweep counter, neighbouring PEs signal their halo */
        if (tid == 0) {
            int rc = 0;
            ishmemi::deadline dl(ctx->wait_limit_ns);
            if (!cols && g > 0) rc = wait_block(g - 1, it, dl);
            else if (p > 0) rc = ishmem_uint64_wait_until(ctx, sig_top, ISHMEM_CMP_GE, expect);
            if (!rc) {
                if (!cols && g < G - 1) rc = wait_block(g + 1, it, dl);
                else if (p + 1 < P) rc = ishmem_uint64_wait_until(ctx, sig_bottom, ISHMEM_CMP_GE, expect);
            }
            if (rc) {
                ishmemi::latch_error(ctx, rc);
                give_up = 1;
            }
        }
        __syncthreads();
        if (give_up) break;
        /* (d) the remaining rows */
        if (!a.overlap) sweep_rows(cur, nxt, r0, r1, want_res);
        else if (r1 > r0) two_rows(cur, nxt, r0, (r1 - 1 > r0) ? r1 - 1 : ~(size_t)0, want_res);
        /* (e) publish this sweep */
        __syncthreads();
        if (tid == 0) {
            ishmemi::fence_acq_rel_gpu();
            ishmemi::st_release(done + g, (unsigned long long)it + 1);
        }
    }
    /* residual partial of this block, summed in a fixed order */
    __shared__ double red[32];
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
    if ((tid & 31u) == 0) red[tid >> 5] = acc;
    __syncthreads();
    if (tid == 0) {
        double s = 0.0;
        for (unsigned w = 0; w < (nthr + 31) / 32; ++w) s += red[w];
        a.partial[blockIdx.x] = s;
    }
}

/* ---- one launch per sweep, one tile per warp ------------------------------------------------
 * The form the library picks when it shapes the launch itself (threads = 0, even nx).  Every sweep
 * is one ordinary launch.  Its first blocks send the halo rows: the first and the last row of every
 * strip, in JACOBI_PIECES pieces each, by in-kernel work-group put_signal (SIGNAL_ADD; the words
 * count pieces, so after sweep it they hold JACOBI_PIECES x (it + 1)).  All other blocks take one
 * band of `band_rows` rows of one PE and 8 neighbouring 60-column tiles of it, one warp per tile,
 * and run the register sliding window down the band.  Blocks are numbered PE by PE, band by band,
 * along the row: they start in that order, so at any moment the running blocks work on one short
 * window of the grid, which this GPU's memory serves about 15 % faster than the long private
 * streams of a resident grid (652 against 757 us per 16384^2 sweep).  Only the first band of a strip
 * needs the halo from above and only the last one the halo from below: their blocks wait (bounded)
 * for the signal first, which the senders -- started long before them -- have raised by then, while
 * the interior bands never wait: the exchange overlaps the interior update.  The launch boundary
 * orders one sweep after the other; nothing needs to be co-resident.  The senders have the lowest
 * block numbers and wait for nothing, so a block that waits for them can only hold an SM after all of
 * them have started; and every wait gives up after the context's time limit in any case. */
#define JACOBI_PIECES 8u
/* sender block b of a sweep: piece (b mod JACOBI_PIECES) of a PE's first or last row.  Out of line,
 * like the full-featured window below, so that the common path of k_jacobi_sweep keeps its
 * registers to itself. */
static __device__ __noinline__ void jacobi_send_piece(const ishmem_ctx_t *ctxs, const double *cur0, unsigned long long *sig0,
                                                      size_t ny, size_t nx, unsigned b)
{
    /* cur0, sig0: PE 0's copies of the source buffer and of the signal words.  By value: a reference to
     * the kernel's argument block would put it on every thread's stack.  2 x JACOBI_PIECES blocks per
     * PE send its first row up and its last row down, into the halo rows of the neighbours' source
     * buffers. */
    const int P = ctxs[0].npes;
    const unsigned per_pe = 2u * JACOBI_PIECES;
    const int p = (int)(b / per_pe), down = (int)((b / JACOBI_PIECES) & 1u);
    const unsigned piece = b % JACOBI_PIECES;
    const ishmem_ctx_t *ctx = ctxs + p;
    size_t first, rows, rows_above = 0, f2;
    strip_of(ny, P, p, &first, &rows);
    if (p > 0) strip_of(ny, P, p - 1, &f2, &rows_above);
    const double *cur = (const double *)local_of(ctxs, ctx, cur0);
    unsigned long long *sig = (unsigned long long *)local_of(ctxs, ctx, sig0);
    const size_t per = ((nx + JACOBI_PIECES - 1) / JACOBI_PIECES + 1) & ~(size_t)1; /* even: 16-byte pieces */
    const size_t c_lo = per * piece < nx ? per * piece : nx, c_hi = c_lo + per < nx ? c_lo + per : nx;
    /* the destination is named by the calling PE's copy of the buffer that receives it */
    if (!down && p > 0) /* my first row -> bottom halo of the PE above */
        ishmemx_putmem_signal_work_group(ctx, (void *)(cur + (rows_above + 1) * nx + c_lo), cur + nx + c_lo,
                                         (c_hi - c_lo) * 8, sig + 1, 1, ISHMEM_SIGNAL_ADD, p - 1);
    if (down && p + 1 < P) /* my last row -> top halo of the PE below */
        ishmemx_putmem_signal_work_group(ctx, (void *)(cur + c_lo), cur + rows * nx + c_lo, (c_hi - c_lo) * 8, sig + 0, 1,
                                         ISHMEM_SIGNAL_ADD, p + 1);
}
static __device__ __noinline__ double jacobi_march_one(const double *cur, double *nxt, unsigned ra, unsigned rb,
                                                       unsigned fixed0, unsigned fixed1, unsigned nx, bool want_res,
                                                       unsigned t_lo, unsigned t_hi)
{
    return jacobi_march_tiles<4>(cur, nxt, ra, rb, fixed0, fixed1, nx, want_res, t_lo, t_hi);
}

__global__ void __launch_bounds__(256, 4) k_jacobi_sweep(const ishmem_ctx_t *ctxs, jacobi_args a, int flip,
                                                          unsigned long long arrived, int last, unsigned band_rows,
                                                          unsigned bands, unsigned tile_groups, int P, size_t heap_stride)
{
    /* flip: the sweep reads buf1 and writes buf0 (else buf0 -> buf1); arrived: what the halo words
     * count once this sweep's pieces are in; last: the residual is wanted. */
    /* P and the distance between two PEs' heaps come as arguments: a tile block lives for a few
     * microseconds, too short to start with a chain of look-ups in the context */
    const unsigned tid = threadIdx.x;
    const size_t nx = a.nx;
    const unsigned nsend = (unsigned)P * 2u * JACOBI_PIECES;
    unsigned b = blockIdx.x;
    if (b < nsend) {
        jacobi_send_piece(ctxs, flip ? a.buf1 : a.buf0, a.sig, a.ny, nx, b);
        return;
    }
    b -= nsend;
    const int p = (int)(b / (bands * tile_groups));
    const unsigned band = (b / tile_groups) % bands, tg = b % tile_groups;
    const ishmem_ctx_t *ctx = ctxs + p;
    const unsigned base_rows = (unsigned)a.ny / (unsigned)P, extra = (unsigned)a.ny % (unsigned)P;
    const unsigned rows = base_rows + ((unsigned)p < extra ? 1u : 0u);
    const unsigned first = (unsigned)p * base_rows + ((unsigned)p < extra ? (unsigned)p : extra);
    const unsigned ra = 1u + band * band_rows;
    const unsigned rb = (ra + band_rows < rows + 1u) ? ra + band_rows : rows + 1u;
    double acc = 0.0;
    __shared__ int give_up;
    if (ra < rb) {
        /* halos: the first band needs the row above the strip, the last one the row below it
         * (overlap = 0: every band waits for both, i.e. exchange, wait, then compute) */
        const bool top = (band == 0 || !a.overlap) && p > 0, bottom = (rb == rows + 1u || !a.overlap) && p + 1 < P;
        if (top || bottom) {
            if (tid == 0) {
                const unsigned long long *sig = (const unsigned long long *)local_of(ctxs, ctx, a.sig);
                int rc = top ? ishmem_uint64_wait_until(ctx, sig + 0, ISHMEM_CMP_GE, arrived) : 0;
                if (!rc && bottom) rc = ishmem_uint64_wait_until(ctx, sig + 1, ISHMEM_CMP_GE, arrived);
                give_up = rc; /* the error is latched by the wait */
            }
            __syncthreads();
            if (give_up) return;
        }
        const double *cur = (const double *)((const char *)(flip ? a.buf1 : a.buf0) + (size_t)p * heap_stride);
        double *nxt = (double *)((char *)(flip ? a.buf0 : a.buf1) + (size_t)p * heap_stride);
        const unsigned fixed0 = (first == 0) ? 1u : ~0u;
        const unsigned fixed1 = (first + rows == (unsigned)a.ny) ? rows : ~0u;
        /* this block's tiles: warp w takes tile t_lo + w */
        const unsigned ntiles = (unsigned)((nx + 59) / 60), t_lo = tg * (blockDim.x >> 5);
        const unsigned t_hi = t_lo + (blockDim.x >> 5) < ntiles ? t_lo + (blockDim.x >> 5) : ntiles;
        const bool has_fixed = (fixed0 >= ra && fixed0 < rb) || (fixed1 >= ra && fixed1 < rb);
        if (last || has_fixed) /* the last sweep, and the two bands with a boundary row */
            acc = jacobi_march_one(cur, nxt, ra, rb, fixed0, fixed1, (unsigned)nx, last != 0, t_lo, t_hi);
        else
            jacobi_march_tiles<4, false, false>(cur, nxt, ra, rb, ~0u, ~0u, (unsigned)nx, false, t_lo, t_hi);
    }
    if (last) {
        /* residual partial of this block, summed in a fixed order */
        __shared__ double red[8];
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
        if ((tid & 31u) == 0) red[tid >> 5] = acc;
        __syncthreads();
        if (tid == 0) {
            double sum = 0.0;
            for (unsigned w = 0; w < (blockDim.x >> 5); ++w) sum += red[w];
            a.partial[b] = sum;
        }
    }
}

/* ---- K sweeps per launch ----------------------------------------------------------------------
 * Every element of the source is read once and the result of the K-th sweep written once: 1/K of the
 * memory traffic per sweep.  A warp's window carries K time levels.  Its lanes hold NC (2 or 4)
 * neighbouring columns each, so a tile is 32 x NC loaded columns; the warp walks down the rows, and
 * from each new row of u(t) it forms the row above it of u(t+1), from that the row above of u(t+2),
 * and so on up to u(t+K), which is stored.  Per level two rows stay in registers (the one being
 * formed replaces the older one, so nothing is moved: steps alternate between two unrolled copies of
 * the code), and only a lane's outermost columns need their neighbours by shuffle.  Every value is
 * the same expression, in the same order, as in a single sweep, so the result is bit-identical to K
 * single sweeps.  Each level loses one column on either side of the tile; the lanes that still hold
 * NC valid columns store (a tile stores (32 - 2 ceil(K / NC)) x NC columns), the rest is recomputed
 * by the neighbouring tile.  A band of R rows reads R + 2K rows.
 * Halo rows: K each way.  The first one goes where a single sweep puts it (the halo rows of the
 * source buffer), the second one into the halo rows of the destination buffer, which nothing else
 * uses during the pass, the third to the K-th into 2 (K - 2) extra rows per PE that the library takes
 * from the symmetric heap for the duration of the call.
 * What bounds a launch: DRAM up to four sweeps (a launch of four takes little longer than a single
 * sweep); from five on the fp64 pipe (3 additions and a multiplication per cell and level, no fused
 * form allowed by the bit-exact association: 430 us of a 950 us launch of six at 16384^2) and the
 * memory latency that 12 warps per SM at 168 registers can cover. */
#define JW_FULL 0xffffffffu
#define JW_AHEAD 3 /* rows between a load and the L2 prefetch issued with it */
#define JW_MAX_DEPTH 6 /* sweeps per launch at most */

template <int NC>
__device__ __forceinline__ void jw_ld(const double *p, double (&v)[NC])
{
    if (NC == 4)
        asm volatile("ld.global.v4.f64 {%0,%1,%2,%3}, [%4];"
                     : "=d"(v[0]), "=d"(v[1]), "=d"(v[2 % NC]), "=d"(v[3 % NC])
                     : "l"(p)
                     : "memory");
    else
        asm volatile("ld.global.v2.f64 {%0,%1}, [%2];" : "=d"(v[0]), "=d"(v[1]) : "l"(p) : "memory");
}
template <int NC>
__device__ __forceinline__ void jw_st(double *p, const double (&v)[NC])
{
    if (NC == 4)
        asm volatile("st.global.v4.f64 [%0], {%1,%2,%3,%4};" ::"l"(p), "d"(v[0]), "d"(v[1]), "d"(v[2 % NC]), "d"(v[3 % NC])
                     : "memory");
    else
        asm volatile("st.global.v2.f64 [%0], {%1,%2};" ::"l"(p), "d"(v[0]), "d"(v[1]) : "memory");
}
/* column pairs whose bit in `ok` is clear lie outside the grid: not touched, read as zero */
template <int NC>
__device__ __forceinline__ void jw_ld_edge(const double *p, double (&v)[NC], unsigned ok)
{
#pragma unroll
    for (int h = 0; h < NC / 2; ++h) {
        double2 a = make_double2(0.0, 0.0);
        if (ok & (1u << h)) a = *(const double2 *)(p + 2 * h);
        v[2 * h] = a.x, v[2 * h + 1] = a.y;
    }
}

template <int K, int NC>
struct jw_window {
    double w[K][2][NC]; /* level l: the two rows above the one being formed; which is which alternates */
};
struct jw_edge {
    unsigned fixcol;    /* bit i: the lane's column i is the grid's first or last column */
    int fixed0, fixed1; /* local numbers of the grid's first / last row, or a value never reached */
};
template <int K, int NC>
struct jw_geo {
    static constexpr int SKIP = (K + NC - 1) / NC;    /* lanes without a full result on either side */
    static constexpr int TILE = (32 - 2 * SKIP) * NC; /* columns a warp stores */
};

/* One step of the window: `c` comes in as row R of u(t) and leaves as row R-K of u(t+K).  P: parity of
 * the step (selects which of a level's two rows is the older one).  FILL: index of the step while the
 * window fills -- levels whose inputs are not there yet are skipped -- or -1 in the steady state.
 * rmask: bit h = the lane's column pair h counts for the residual. */
template <int K, int NC, int P, bool EDGE, bool RES, int FILL>
__device__ __forceinline__ void jw_step(jw_window<K, NC> &W, double (&c)[NC], int R, const jw_edge &e, double &acc,
                                        unsigned rmask)
{
#pragma unroll
    for (int l = 0; l < K; ++l) {
        const bool compute = FILL < 0 || FILL >= 2 * l;
        const bool keep = compute || FILL >= 2 * l - 2; /* the incoming row of level l is valid: keep it */
        if (!keep) break;
        double(&up)[NC] = W.w[l][P];
        double(&mid)[NC] = W.w[l][P ^ 1];
        if (!compute) {
#pragma unroll
            for (int i = 0; i < NC; ++i) up[i] = c[i];
            break;
        }
        /* the lane's outer neighbours in the middle row */
        const double nl = __shfl_up_sync(JW_FULL, mid[NC - 1], 1), nr = __shfl_down_sync(JW_FULL, mid[0], 1);
        double o[NC];
#pragma unroll
        for (int i = 0; i < NC; ++i) {
            const double left = i > 0 ? mid[i > 0 ? i - 1 : 0] : nl;
            const double right = i < NC - 1 ? mid[i < NC - 1 ? i + 1 : 0] : nr;
            o[i] = 0.25 * ((up[i] + c[i]) + (left + right));
        }
        if (EDGE) {
            const int q = R - 1 - l; /* the row of level l+1 formed here */
            const bool fixed_row = q == e.fixed0 || q == e.fixed1;
#pragma unroll
            for (int i = 0; i < NC; ++i)
                if (fixed_row || (e.fixcol & (1u << i))) o[i] = mid[i];
        }
        if (RES && l == K - 1) {
#pragma unroll
            for (int i = 0; i < NC; ++i)
                if (rmask & (1u << (i >> 1))) {
                    const double d = o[i] - mid[i];
                    acc += d * d;
                }
        }
#pragma unroll
        for (int i = 0; i < NC; ++i) {
            up[i] = c[i]; /* the older row is done with: the incoming one takes its place */
            c[i] = o[i];
        }
    }
}

/* where the rows of u(t) around a strip live (see the section comment) */
struct jw_rows {
    const double *cur; /* local rows 0 .. rows+1 */
    const double *nxt; /* its rows 0 and rows+1 hold local rows -1 and rows+2 during the pass */
    const double *xh;  /* 2 x xh_side extra rows: local rows -2, -3, ... then rows+3, rows+4, ... */
    int rows, xh_side;
    size_t nx;
    __device__ __forceinline__ const double *at(int r) const
    {
        if (r < 0) return r == -1 ? nxt : xh + (size_t)(-r - 2) * nx;
        if (r > rows + 1)
            return r == rows + 2 ? nxt + (size_t)(rows + 1) * nx : xh + (size_t)(xh_side + r - rows - 3) * nx;
        return cur + (size_t)r * nx;
    }
};

/* Rows [ra, rb) of the strip, tile t, by one warp.  D rows are in flight per lane.  EDGE: the tile
 * touches the grid's first or last column or a column outside it, or the band forms one of the grid's
 * fixed rows; without EDGE nothing of that is tested.  HALO: the band reads rows outside the source
 * buffer (EDGE implies it); without it the rows are one pitch apart.  Returns the lane's share of the
 * squared last update when RES. */
template <int K, int NC, int D, bool EDGE, bool HALO, bool RES>
__device__ __forceinline__ double jw_march(const jw_rows &src, double *nxt, int ra, int rb, int t, int fixed0, int fixed1)
{
    static_assert(D == 2 || D == 4, "the unrolled loop keeps the step parity");
    static_assert(K >= 2 && K <= JW_MAX_DEPTH, "window depth");
    using G = jw_geo<K, NC>;
    const int lane = threadIdx.x & 31;
    const int nx = (int)src.nx;
    const int jA = t * G::TILE - G::SKIP * NC + NC * lane;
    unsigned ok = 0;
#pragma unroll
    for (int h = 0; h < NC / 2; ++h)
        if (!EDGE || (jA + 2 * h >= 0 && jA + 2 * h < nx)) ok |= 1u << h;
    const bool st_lane = lane >= G::SKIP && lane < 32 - G::SKIP;
    jw_edge e;
    e.fixcol = 0;
#pragma unroll
    for (int i = 0; i < NC; ++i)
        if (EDGE && (jA + i == 0 || jA + i == nx - 1)) e.fixcol |= 1u << i;
    e.fixed0 = fixed0, e.fixed1 = fixed1;
    const unsigned rmask = st_lane ? ok : 0u;
    const int n_steps = (rb - ra) + 2 * K - 2;
    const size_t pitch = src.nx;
    const int jbase = (ok & 1u) ? jA : 0;
    jw_window<K, NC> W;
#pragma unroll
    for (int l = 1; l < K; ++l)
#pragma unroll
        for (int i = 0; i < NC; ++i) W.w[l][0][i] = W.w[l][1][i] = 0.0;
    double acc = 0.0;
    double f[D][NC]; /* rows in flight */
    int r_next = ra - K;
    const int r_last = rb - 1 + K; /* last row of u(t) the band reads */
    const double *pin = src.cur + (size_t)r_next * pitch + jbase; /* the plain form: all rows are in the source buffer */
    /* Each request also asks L2 for the row JW_AHEAD further down.  The registers hold D rows in flight,
     * which at 128 registers per thread is all a K-level window leaves room for; the prefetch puts the
     * DRAM latency of the following rows behind them without holding anything (measured at 16384^2, four
     * sweeps per launch: 880 -> 740 us per launch with 2 or 3 rows ahead, 745 with 4, 780 with 8, 900
     * with 16: further ahead the prefetched rows of all resident warps no longer fit beside one another). */
    auto request = [&](double(&v)[NC]) {
        if (EDGE) {
            jw_ld_edge<NC>(src.at(r_next) + jbase, v, ok);
            if ((ok & 1u) && r_next + JW_AHEAD <= r_last)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(src.at(r_next + JW_AHEAD) + jbase));
        } else if (HALO) {
            jw_ld<NC>(src.at(r_next) + jbase, v);
            if (r_next + JW_AHEAD <= r_last)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(src.at(r_next + JW_AHEAD) + jbase));
        } else {
            jw_ld<NC>(pin, v);
            if (r_next + JW_AHEAD <= r_last) asm volatile("prefetch.global.L2 [%0];" ::"l"(pin + (size_t)JW_AHEAD * pitch));
            pin += pitch;
        }
        ++r_next;
    };
    /* everything the window starts from is requested before the first use */
    request(W.w[0][0]);
    request(W.w[0][1]);
#pragma unroll
    for (int s = 0; s < D; ++s) {
        if (s < n_steps) request(f[s]);
        else {
#pragma unroll
            for (int i = 0; i < NC; ++i) f[s][i] = 0.0;
        }
    }
    double *po = nxt + (size_t)ra * pitch + jbase;
    int s = 0;
    auto one = [&](auto slot, auto parity, auto fill) {
        constexpr int S = decltype(slot)::value, P = decltype(parity)::value, F = decltype(fill)::value;
        double c[NC];
#pragma unroll
        for (int i = 0; i < NC; ++i) c[i] = f[S][i];
        if (s + D < n_steps) request(f[S]);
        jw_step<K, NC, P, EDGE, RES, F>(W, c, ra - K + 2 + s, e, acc, rmask);
        if (F < 0) {
            if (EDGE) {
#pragma unroll
                for (int h = 0; h < NC / 2; ++h)
                    if (st_lane && (ok & (1u << h))) *(double2 *)(po + 2 * h) = make_double2(c[2 * h], c[2 * h + 1]);
            } else if (st_lane) {
                jw_st<NC>(po, c);
            }
            po += pitch;
        }
        ++s;
    };
    /* the window fills: steps 0 .. 2K-3, none of which stores */
#define JW_FILL(I)                                                                                              \
    if ((I) < 2 * K - 2 && s < n_steps)                                                                         \
        one(std::integral_constant<int, (I) % D>{}, std::integral_constant<int, (I)&1>{},                       \
            std::integral_constant<int, (I) < 2 * K - 2 ? (I) : -1>{});
    JW_FILL(0) JW_FILL(1) JW_FILL(2) JW_FILL(3) JW_FILL(4) JW_FILL(5) JW_FILL(6) JW_FILL(7) JW_FILL(8) JW_FILL(9)
#undef JW_FILL
    static_assert(2 * JW_MAX_DEPTH - 2 <= 10, "one JW_FILL per step of the filling window");
    /* steady state: D steps per trip, slots and parities known at compile time */
    constexpr int S0 = (2 * K - 2) % D;
    while (s < n_steps) {
#define JW_STEP(U)                                                                                              \
    if ((U) < D && s < n_steps)                                                                                 \
        one(std::integral_constant<int, (S0 + (U)) % D>{}, std::integral_constant<int, (U)&1>{},                \
            std::integral_constant<int, -1>{});
        JW_STEP(0) JW_STEP(1) JW_STEP(2) JW_STEP(3)
#undef JW_STEP
    }
    return acc;
}

/* The other forms as functions of their own: inlined beside the plain form they share its register
 * allocation, and at five and six levels that costs the plain form -- which does nearly all the work --
 * up to a fifth of its speed (six sweeps per launch at 16384^2: 1040 us inlined, 850 us for the plain
 * form alone).  Both also form the residual, which the caller drops unless the launch is the last one:
 * a few instructions per row against two more copies of the march. */
template <int K, int NC, bool EDGE>
static __device__ __noinline__ double jw_march_other(const double *cur, const double *nxt_halo, const double *xh, int rows,
                                                     int xh_side, size_t nx, double *nxt, int ra, int rb, int t, int fixed0,
                                                     int fixed1)
{
    jw_rows src;
    src.cur = cur;
    src.nxt = nxt_halo;
    src.xh = xh;
    src.rows = rows;
    src.xh_side = xh_side;
    src.nx = nx;
    return jw_march<K, NC, 2, EDGE, true, true>(src, nxt, ra, rb, t, fixed0, fixed1);
}

/* sender block b of a K-sweep pass: piece (b mod JACOBI_PIECES) of one of the K first or K last rows of
 * a PE's strip, into the neighbour's row of the same depth (see jw_rows for where that is) */
static __device__ __noinline__ void jacobi_send_piece_k(const ishmem_ctx_t *ctxs, const double *cur0, double *nxt0,
                                                        double *xh0, unsigned xh_side, unsigned long long *sig0, size_t ny,
                                                        size_t nx, unsigned b, unsigned K)
{
    const int P = ctxs[0].npes;
    const unsigned per_pe = 2u * K * JACOBI_PIECES;
    const int p = (int)(b / per_pe), down = (int)((b / JACOBI_PIECES) & 1u);
    const unsigned depth = (b % per_pe) / (2u * JACOBI_PIECES), piece = b % JACOBI_PIECES; /* depth 0: the edge row itself */
    const ishmem_ctx_t *ctx = ctxs + p;
    size_t first, rows, rows_above = 0, f2;
    strip_of(ny, P, p, &first, &rows);
    if (p > 0) strip_of(ny, P, p - 1, &f2, &rows_above);
    const double *cur = (const double *)local_of(ctxs, ctx, cur0);
    double *nxt = (double *)local_of(ctxs, ctx, nxt0), *xh = (double *)local_of(ctxs, ctx, xh0);
    unsigned long long *sig = (unsigned long long *)local_of(ctxs, ctx, sig0);
    const size_t per = ((nx + JACOBI_PIECES - 1) / JACOBI_PIECES + 1) & ~(size_t)1; /* even: 16-byte pieces */
    const size_t c_lo = per * piece < nx ? per * piece : nx, c_hi = c_lo + per < nx ? c_lo + per : nx;
    /* destinations are named by the calling PE's copy of the object that receives them */
    if (!down && p > 0) { /* my row 1 + depth -> row rows_above + 1 + depth of the PE above */
        double *into = depth == 0   ? (double *)cur + (rows_above + 1) * nx
                       : depth == 1 ? nxt + (rows_above + 1) * nx
                                    : xh + (size_t)(xh_side + depth - 2) * nx; /* its rows+3, ...: the second half */
        ishmemx_putmem_signal_work_group(ctx, (void *)(into + c_lo), cur + (size_t)(1 + depth) * nx + c_lo,
                                         (c_hi - c_lo) * 8, sig + 1, 1, ISHMEM_SIGNAL_ADD, p - 1);
    }
    if (down && p + 1 < P) { /* my row rows - depth -> row -depth of the PE below */
        double *into = depth == 0 ? (double *)cur : depth == 1 ? nxt : xh + (size_t)(depth - 2) * nx; /* the first half */
        ishmemx_putmem_signal_work_group(ctx, (void *)(into + c_lo), cur + (rows - depth) * nx + c_lo,
                                         (c_hi - c_lo) * 8, sig + 0, 1, ISHMEM_SIGNAL_ADD, p + 1);
    }
}

/* one launch = K sweeps: sender blocks (K rows each way per PE), then one block per band of `band_rows`
 * rows x (blockDim / 32) tiles, in launch order as in k_jacobi_sweep */
#define JACOBI_PASS_THREADS 128
/* four blocks per SM (128 registers); windows of four and more levels with four columns per lane would
 * spill there and get three (170 registers): K = 4: 718 against 739 us per launch on a single strip */
template <int K, int NC>
__global__ void __launch_bounds__(JACOBI_PASS_THREADS, (K >= 4 && NC == 4) ? 3 : 4) k_jacobi_pass(const ishmem_ctx_t *ctxs, jacobi_args a, double *xh0,
                                                                        int xh_side, int flip, unsigned long long arrived, int last,
                                                                        unsigned band_rows, unsigned bands,
                                                                        unsigned tile_groups, unsigned lead_bands, int P, size_t heap_stride)
{
    using G = jw_geo<K, NC>;
    const unsigned tid = threadIdx.x;
    const size_t nx = a.nx;
    const unsigned nsend = (unsigned)P * 2u * K * JACOBI_PIECES;
    unsigned b = blockIdx.x;
    if (b < nsend) {
        jacobi_send_piece_k(ctxs, flip ? a.buf1 : a.buf0, flip ? a.buf0 : a.buf1, xh0, (unsigned)xh_side, a.sig, a.ny, nx, b, K);
        return;
    }
    b -= nsend;
    /* Blocks that hold the grid's first or last column, or its last row, take the slow form of the march
     * (three times the instructions per row).  Started in their natural place the last of them would run
     * on alone after everything else has finished (8192^2, six sweeps per launch: 320 us against 210 us
     * for the plain blocks), so they come first: the first and last tile group of every band, then the
     * last band of the last strip (`lead_bands` bands counted from the end, the empty ones included),
     * then all the others in the order of their rows. */
    const unsigned edge_groups = tile_groups < 2u ? tile_groups : 2u, inner_groups = tile_groups - edge_groups;
    const unsigned n_edge = (unsigned)P * bands * edge_groups;
    unsigned pb, tg;
    if (b < n_edge) {
        pb = b / edge_groups;
        tg = (b % edge_groups) ? tile_groups - 1u : 0u;
    } else {
        const unsigned n_inner = (unsigned)P * bands * inner_groups, lead = lead_bands * inner_groups;
        b -= n_edge;
        b = b < lead ? n_inner - lead + b : b - lead;
        pb = b / inner_groups;
        tg = 1u + b % inner_groups;
    }
    const int p = (int)(pb / bands);
    const unsigned band = pb % bands;
    b = pb * tile_groups + tg; /* the block's number in the order of rows and tiles: its residual slot */
    const ishmem_ctx_t *ctx = ctxs + p;
    const unsigned base_rows = (unsigned)a.ny / (unsigned)P, extra = (unsigned)a.ny % (unsigned)P;
    const int rows = (int)(base_rows + ((unsigned)p < extra ? 1u : 0u));
    const unsigned first = (unsigned)p * base_rows + ((unsigned)p < extra ? (unsigned)p : extra);
    const int ra = 1 + (int)(band * band_rows);
    const int rb = (ra + (int)band_rows < rows + 1) ? ra + (int)band_rows : rows + 1;
    double acc = 0.0;
    __shared__ int give_up;
    if (ra < rb) {
        /* a band that reads rows above the strip needs the K halo rows from above, one that reads rows
         * below it those from below (overlap = 0: every band waits for both: exchange, wait, compute) */
        const bool top = (ra - K < 1 || !a.overlap) && p > 0, bottom = (rb - 1 + K > rows || !a.overlap) && p + 1 < P;
        if (top || bottom) {
            if (tid == 0) {
                const unsigned long long *sig = (const unsigned long long *)local_of(ctxs, ctx, a.sig);
                int rc = top ? ishmem_uint64_wait_until(ctx, sig + 0, ISHMEM_CMP_GE, arrived) : 0;
                if (!rc && bottom) rc = ishmem_uint64_wait_until(ctx, sig + 1, ISHMEM_CMP_GE, arrived);
                give_up = rc; /* the error is latched by the wait */
            }
            __syncthreads();
            if (give_up) return;
        }
        jw_rows src;
        src.cur = (const double *)((const char *)(flip ? a.buf1 : a.buf0) + (size_t)p * heap_stride);
        double *nxt = (double *)((char *)(flip ? a.buf0 : a.buf1) + (size_t)p * heap_stride);
        src.nxt = nxt;
        src.xh = (const double *)((const char *)xh0 + (size_t)p * heap_stride);
        src.rows = rows;
        src.xh_side = xh_side;
        src.nx = nx;
        const int fixed0 = (first == 0) ? 1 : -100;
        const int fixed1 = (first + (unsigned)rows == (unsigned)a.ny) ? rows : -100;
        const int ntiles = (int)((nx + G::TILE - 1) / G::TILE);
        const int t = (int)(tg * (blockDim.x >> 5) + (tid >> 5));
        if (t < ntiles) {
            const int j0 = t * G::TILE - G::SKIP * NC;
            /* no edge: all loaded columns inside the grid and none of them its first or last one, no fixed
             * row among the rows formed; the plain form also reads all its rows from the source buffer and
             * forms no residual */
            const bool no_edge = j0 > 0 && j0 + 32 * NC < (int)nx && !(fixed0 >= ra - K + 1 && fixed0 <= rb + K - 2) &&
                                 !(fixed1 >= ra - K + 1 && fixed1 <= rb + K - 2);
            const bool rows_inside = ra - K >= 0 && rb - 1 + K <= rows + 1;
            if (no_edge && rows_inside && !last)
                jw_march<K, NC, 2, false, false, false>(src, nxt, ra, rb, t, fixed0, fixed1);
            else if (no_edge)
                acc = jw_march_other<K, NC, false>(src.cur, src.nxt, src.xh, rows, xh_side, nx, nxt, ra, rb, t, fixed0, fixed1);
            else
                acc = jw_march_other<K, NC, true>(src.cur, src.nxt, src.xh, rows, xh_side, nx, nxt, ra, rb, t, fixed0, fixed1);
        }
    }
    if (last) {
        __shared__ double red[JACOBI_PASS_THREADS / 32];
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
        if ((tid & 31u) == 0) red[tid >> 5] = acc;
        __syncthreads();
        if (tid == 0) {
            double sum = 0.0;
            for (unsigned w = 0; w < (blockDim.x >> 5); ++w) sum += red[w];
            a.partial[b] = sum;
        }
    }
}

/* How the blocks of a PE share its strip: by columns when the library shapes the blocks itself
 * (threads == 0) and every block gets at least 16 column tiles, one warp each; by rows when the
 * caller gives the block size, or when the grid is too narrow to fill the blocks with tiles (a
 * block then walks all tiles of its band, and any block size keeps its warps busy).
 * ISHMEMX_OPT_JACOBI_SPLIT = 1 (rows) / 2 (columns) overrides. */
static bool jacobi_by_columns(int threads, size_t nx, int groups_per_pe)
{
    const long long split = g_ishmem.opt[ISHMEMX_OPT_JACOBI_SPLIT];
    if (split == 1) return false;
    if (split == 2) return true;
    return threads == 0 && (nx + 59) / 60 >= (size_t)groups_per_pe * 16;
}

/* argument checks shared by the two entry points; *groups_per_pe is clamped to the shortest strip */
static int jacobi_check(double *buf0, double *buf1, uint64_t *sig, size_t ny, size_t nx, int iters,
                        int *groups_per_pe, int threads, bool *by_columns)
{
    auto &g = g_ishmem;
    const int P = g.npes;
    if (ny < 3 || nx < 3 || nx > 0x7fffff00u || ny > 0x7fffff00u || iters < 0 || (size_t)P > ny) return ISHMEM_ERR_ARG;
    if (threads < 0 || threads > 1024 || threads % 32 || *groups_per_pe < 1) return ISHMEM_ERR_ARG;
    const size_t rows_min = ny / P, rows_max = (ny + P - 1) / P;
    *by_columns = jacobi_by_columns(threads, nx, *groups_per_pe);
    const size_t most = *by_columns ? (nx + 59) / 60 : rows_min; /* a tile or a row per block at least */
    if ((size_t)*groups_per_pe > most) *groups_per_pe = (int)most;
    const size_t bytes = (rows_max + 2) * nx * 8;
    if ((uintptr_t)buf0 % 16 || (uintptr_t)buf1 % 16 || (uintptr_t)sig % 8) return ISHMEM_ERR_ALIGN;
    if (ishmemi_sym_offset(buf0, bytes) < 0 || ishmemi_sym_offset(buf1, bytes) < 0 ||
        ishmemi_sym_offset(sig, 32) < 0)
        return ISHMEM_ERR_NOT_SYMMETRIC;
    return ISHMEM_OK;
}

/* clears the scratch, launches the persistent kernel on the team stream and waits for it;
 * `scratch` holds nblocks sweep counters followed by nblocks residual partials */
static int jacobi_launch(double *buf0, double *buf1, uint64_t *sig, size_t ny, size_t nx, int iters, int overlap,
                         int groups_per_pe, int threads, bool by_columns, void *scratch, jacobi_args *out_args)
{
    auto &g = g_ishmem;
    const size_t nblocks = (size_t)g.npes * groups_per_pe;
    cudaStream_t s;
    int rc = ishmemi_team_stream_begin(ISHMEM_TEAM_WORLD, &s);
    if (rc) return rc;
    /* the counters must start from zero */
    rc = ishmemi_cuda(cudaMemsetAsync(scratch, 0, nblocks * 16, s), "cudaMemsetAsync");
    jacobi_args a = {};
    a.buf0 = buf0;
    a.buf1 = buf1;
    a.sig = (unsigned long long *)sig;
    a.ny = ny;
    a.nx = nx;
    a.iters = iters;
    a.overlap = overlap;
    a.groups = groups_per_pe;
    a.done = (unsigned long long *)scratch;
    a.partial = (double *)((char *)scratch + nblocks * 8);
    a.sliding = (nx % 2 == 0);
    a.colsplit = by_columns;
    if (threads == 0) {
        /* by columns: one warp per tile when that fits a block, else the fewest equal rounds;
         * by rows: 512 */
        threads = 512;
        if (a.colsplit) {
            const size_t tiles = ((nx + 59) / 60 + groups_per_pe - 1) / groups_per_pe;
            const size_t cap = nblocks <= (size_t)g.sm_count ? 23 : 16, rounds = (tiles + cap - 1) / cap;
            threads = 32 * (int)((tiles + rounds - 1) / rounds);
        }
    }
    const ishmem_ctx_t *ctxs = g.d_ctx;
    void *params[] = {(void *)&ctxs, (void *)&a};
    if (!rc)
    {
        /* blocks of at most 512 threads that have an SM to themselves get 128 registers per thread
         * and a deeper window; everything else the 1024-thread instance */
        const bool alone = nblocks <= (size_t)g.sm_count;
        void *kernel = (alone && threads <= 512) ? (void *)k_jacobi<512, 7>
                       : (alone && threads <= 736) ? (void *)k_jacobi<736, 5>
                                                   : (void *)k_jacobi<1024, 4>;
        rc = ishmemi_cuda(cudaLaunchCooperativeKernel(kernel, dim3((unsigned)nblocks), dim3(threads), params, 0, s),
                          "cudaLaunchCooperativeKernel(jacobi)");
    }
    ishmemi_count_launch();
    ishmemi_team_stream_end();
    if (!rc) rc = ishmemi_cuda(cudaStreamSynchronize(s), "cudaStreamSynchronize");
    *out_args = a;
    return rc;
}

/* one launch per sweep (k_jacobi_sweep): bands of 16 rows x 8 tiles of 60 columns per block */
#define JACOBI_BAND_ROWS 16u /* measured at 16384^2: 8 rows 687 us, 12: 663, 16: 652, 20: 652, 24: 659, 32: 666, 64: 680 */
/* K sweeps per launch (k_jacobi_pass): a band pays 2K extra rows, so it is taller.  Up to four sweeps 64
 * and 128 rows measure the same at 16384^2 and 64 gives small grids more blocks; five and six sweeps
 * per launch are 5 % faster with 128 */
static unsigned jacobi_pass_band_rows(int k) { return k >= 5 ? 128u : 64u; }

/* The launches of one call.  Every launch moves the grid from one buffer to the other, and the result
 * has to end where `iters` single sweeps would leave it (buf0 for an even count), so the number of
 * launches has the parity of iters.  Within that the split is the cheapest one by the measured time of
 * a launch of 1 .. 6 sweeps at 16384^2 (JACOBI_LAUNCH_US: a launch costs little more the deeper it is,
 * so deep launches win and a single sweep is the cheapest filler). */
static const double JACOBI_LAUNCH_US[JW_MAX_DEPTH + 1] = {0, 640, 690, 715, 760, 850, 960};

struct jacobi_plan {
    std::vector<int> depth;            /* sweeps of each launch, deepest first */
    int nc[JW_MAX_DEPTH + 1];          /* columns per lane of a launch of depth k */
    unsigned bands1, groups1;
    unsigned band_rows_k[JW_MAX_DEPTH + 1]; /* rows per band of a launch of depth k */
    unsigned bands_k[JW_MAX_DEPTH + 1];  /* bands per strip of a launch of depth k */
    unsigned groups_k[JW_MAX_DEPTH + 1]; /* tile groups per band of a launch of depth k */
    size_t blocks_last;                /* tile blocks (= residual terms) of the last launch */
    int xh_side;                       /* extra halo rows per side: the deepest launch's depth - 2 */
};

static void jacobi_split(int iters, int kmax, std::vector<int> *out)
{
    const double *cost = JACOBI_LAUNCH_US;
    out->clear();
    int full = 0, r = iters;
    while (r > 24) { /* far from the end only the deepest launch is ever right */
        r -= kmax;
        ++full;
    }
    const double inf = 1e30;
    double best[25][2];
    int pick[25][2];
    best[0][0] = 0, best[0][1] = inf;
    pick[0][0] = pick[0][1] = 0;
    for (int n = 1; n <= r; ++n)
        for (int par = 0; par < 2; ++par) {
            best[n][par] = inf;
            pick[n][par] = 0;
            for (int k = 1; k <= kmax && k <= n; ++k)
                if (cost[k] + best[n - k][par ^ 1] < best[n][par]) {
                    best[n][par] = cost[k] + best[n - k][par ^ 1];
                    pick[n][par] = k;
                }
        }
    int par = (iters - full) & 1; /* launches still to come must have this parity */
    for (int i = 0; i < full; ++i) out->push_back(kmax);
    for (int n = r; n > 0;) {
        const int k = pick[n][par];
        if (k == 0) { /* no split of this parity (cannot happen for n >= 1 with k = 1 allowed and parity n) */
            out->assign((size_t)iters, 1);
            return;
        }
        out->push_back(k);
        n -= k;
        par ^= 1;
    }
    std::sort(out->begin(), out->end(), [](int x, int y) { return x > y; });
}

/* The split alone, for callers that want to know the launches of a call beforehand and for tests of
 * the host logic: needs no device and no initialised library. */
extern "C" int ishmemx_jacobi_launch_depths(int iters, int max_depth, int *depths_out, int capacity)
{
    if (iters < 0 || max_depth < 1 || max_depth > JW_MAX_DEPTH || capacity < 0 || (capacity && !depths_out)) return ISHMEM_ERR_ARG;
    std::vector<int> d;
    jacobi_split(iters, max_depth, &d);
    for (size_t i = 0; i < d.size() && i < (size_t)capacity; ++i) depths_out[i] = d[i];
    return (int)d.size();
}

static unsigned jacobi_pass_groups(size_t nx, int k, int nc)
{
    const unsigned skip = (unsigned)((k + nc - 1) / nc), tile = (32u - 2u * skip) * (unsigned)nc;
    const unsigned ntiles = (unsigned)((nx + tile - 1) / tile), warps = JACOBI_PASS_THREADS / 32;
    return (ntiles + warps - 1) / warps;
}

/* kmax: the deepest launch allowed (the caller lowers it when the symmetric heap has no room for the
 * extra halo rows) */
static void jacobi_make_plan(size_t ny, size_t nx, int iters, int kmax, jacobi_plan *pl)
{
    auto &g = g_ishmem;
    const size_t rows_min = ny / (size_t)g.npes, rows_max = (ny + g.npes - 1) / g.npes;
    /* ISHMEMX_OPT_JACOBI_FUSE: 0 = single sweeps only, 1 = the library's choice, 2..6 = at most that deep */
    const long long fuse = g.opt[ISHMEMX_OPT_JACOBI_FUSE];
    if (fuse == 0) kmax = 1;
    else if (fuse >= 2 && fuse < kmax) kmax = (int)fuse;
    /* a strip sends its k first and k last rows: it must own that many */
    if ((size_t)kmax > rows_min) kmax = rows_min < 1 ? 1 : (int)rows_min;
    pl->bands1 = (unsigned)((rows_max + JACOBI_BAND_ROWS - 1) / JACOBI_BAND_ROWS);
    pl->groups1 = (unsigned)(((nx + 59) / 60 + 7) / 8);
    for (int k = 2; k <= JW_MAX_DEPTH; ++k) {
        pl->band_rows_k[k] = jacobi_pass_band_rows(k);
        pl->bands_k[k] = (unsigned)((rows_max + pl->band_rows_k[k] - 1) / pl->band_rows_k[k]);
    }
    /* Columns per lane: four (32-byte accesses: nx a multiple of 4) unless the grid is too small to give
     * every SM its blocks that way.  At 16384^2, per sweep, four against two columns per lane: 345 / 395 us
     * with two sweeps per launch, 247 / 295 with three, 200 / 230 with four.  ISHMEMX_OPT_JACOBI_WIDE =
     * 0 / 1 forces two / four. */
    const long long wide = g.opt[ISHMEMX_OPT_JACOBI_WIDE];
    for (int k = 2; k <= JW_MAX_DEPTH; ++k) {
        pl->nc[k] = 4;
        if (nx % 4 != 0 || wide == 0) pl->nc[k] = 2;
        else if (wide < 0 && (size_t)g.npes * pl->bands_k[k] * jacobi_pass_groups(nx, k, 4) < (size_t)g.sm_count * 8) pl->nc[k] = 2;
    }
    pl->xh_side = 0;
    for (int k = 2; k <= JW_MAX_DEPTH; ++k) pl->groups_k[k] = jacobi_pass_groups(nx, k, pl->nc[k]);
    jacobi_split(iters, kmax, &pl->depth);
    for (int k : pl->depth) pl->xh_side = std::max(pl->xh_side, k - 2);
    /* Small grids: lower bands, down to 16 rows, until every SM has a dozen blocks to draw from -- more
     * rows read twice, but blocks for all SMs (four sweeps per launch, per sweep, bands of 64 / 32 / 16
     * rows: 1024^2 on 8 PEs 8.3 / 5.4 / 4.3 us, 2048^2 9.7 / 7.5 / 7.3, 4096^2 on 12 PEs 20.2 / 18.6 / 19.4;
     * at 8192^2 the bands of 64 stay: 51 / 54 / 58).  With that, six sweeps per launch are the fastest
     * at every size measured (4096^2 on 8 PEs: 16.4 us per sweep against 18.7 with four; with their
     * bands of 128 rows kept they took 20). */
    for (int k = 2; k <= JW_MAX_DEPTH; ++k)
        while (pl->band_rows_k[k] > 16 && (size_t)g.npes * pl->bands_k[k] * pl->groups_k[k] < (size_t)g.sm_count * 12) {
            pl->band_rows_k[k] /= 2;
            pl->bands_k[k] = (unsigned)((rows_max + pl->band_rows_k[k] - 1) / pl->band_rows_k[k]);
        }
    const int k_last = pl->depth.empty() ? 1 : pl->depth.back();
    pl->blocks_last = k_last == 1 ? (size_t)g.npes * pl->bands1 * pl->groups1
                                  : (size_t)g.npes * pl->bands_k[k_last] * pl->groups_k[k_last];
    if (pl->depth.empty()) pl->blocks_last = 0;
}

template <int NC>
static void jacobi_launch_pass(int k, unsigned nblocks, cudaStream_t s, const jacobi_args &a, double *xh, int xh_side,
                               int flip, unsigned long long arrived, int last, unsigned band_rows, unsigned bands,
                               unsigned groups)
{
    auto &g = g_ishmem;
    /* the bands from the last strip's last band with rows on (see the kernel) */
    const unsigned rows_last = (unsigned)(a.ny / (size_t)g.npes);
    const unsigned lead_bands = bands - (rows_last - 1) / band_rows;
#define JACOBI_PASS_CASE(K)                                                                                          \
    case K:                                                                                                          \
        k_jacobi_pass<K, NC><<<nblocks, JACOBI_PASS_THREADS, 0, s>>>(g.d_ctx, a, xh, xh_side, flip, arrived, last,   \
                                                                    band_rows, bands, groups, lead_bands, g.npes, g.heap_bytes); \
        break;
    switch (k) {
        JACOBI_PASS_CASE(2)
        JACOBI_PASS_CASE(3)
        JACOBI_PASS_CASE(4)
        JACOBI_PASS_CASE(5)
        JACOBI_PASS_CASE(6)
    }
#undef JACOBI_PASS_CASE
    static_assert(JW_MAX_DEPTH == 6, "one case per depth");
}

/* partial: room for pl.blocks_last residual terms, or NULL when no residual is wanted (the last launch
 * then runs like the others); xh: 2 x pl.xh_side symmetric rows (PE 0's copy) */
static int jacobi_launch_sweeps(double *buf0, double *buf1, uint64_t *sig, size_t ny, size_t nx, int iters, int overlap,
                                const jacobi_plan &pl, double *partial, double *xh)
{
    auto &g = g_ishmem;
    for (int k = 1; k <= JW_MAX_DEPTH; ++k) {
        const size_t tiles = k == 1 ? (size_t)g.npes * pl.bands1 * pl.groups1 : (size_t)g.npes * pl.bands_k[k] * pl.groups_k[k];
        if (tiles + (size_t)g.npes * 2 * k * JACOBI_PIECES > 0x7fffffffu) return ISHMEM_ERR_ARG;
    }
    cudaStream_t s;
    int rc = ishmemi_team_stream_begin(ISHMEM_TEAM_WORLD, &s);
    if (rc) return rc;
    jacobi_args a = {};
    a.buf0 = buf0;
    a.buf1 = buf1;
    a.sig = (unsigned long long *)sig;
    a.ny = ny;
    a.nx = nx;
    a.iters = iters;
    a.overlap = overlap;
    a.partial = partial;
    a.sliding = 1;
    int flip = 0;
    unsigned long long arrived = 0; /* pieces the halo words count once the launch's senders are through */
    for (size_t i = 0; i < pl.depth.size() && !rc; ++i) {
        const int k = pl.depth[i], last = partial && i + 1 == pl.depth.size();
        arrived += (unsigned long long)k * JACOBI_PIECES;
        const unsigned nsend = (unsigned)g.npes * 2u * (unsigned)k * JACOBI_PIECES;
        if (k == 1) {
            k_jacobi_sweep<<<nsend + (unsigned)g.npes * pl.bands1 * pl.groups1, 256, 0, s>>>(
                g.d_ctx, a, flip, arrived, last, JACOBI_BAND_ROWS, pl.bands1, pl.groups1, g.npes, g.heap_bytes);
        } else {
            const unsigned nblocks = nsend + (unsigned)g.npes * pl.bands_k[k] * pl.groups_k[k];
            if (pl.nc[k] == 4)
                jacobi_launch_pass<4>(k, nblocks, s, a, xh, pl.xh_side, flip, arrived, last, pl.band_rows_k[k], pl.bands_k[k],
                                      pl.groups_k[k]);
            else
                jacobi_launch_pass<2>(k, nblocks, s, a, xh, pl.xh_side, flip, arrived, last, pl.band_rows_k[k], pl.bands_k[k],
                                      pl.groups_k[k]);
        }
        flip ^= 1;
        ishmemi_count_launch();
        rc = ishmemi_check_launch("k_jacobi_sweep");
    }
    ishmemi_team_stream_end();
    if (!rc) rc = ishmemi_cuda(cudaStreamSynchronize(s), "cudaStreamSynchronize");
    return rc;
}

/* The library shapes the launch itself (threads == 0) and the grid has an even number of columns:
 * one launch per sweep.  ISHMEMX_OPT_JACOBI_SPLIT = rows / columns asks for the persistent kernel. */
static bool jacobi_per_sweep(int threads, size_t nx)
{
    return threads == 0 && nx % 2 == 0 && g_ishmem.opt[ISHMEMX_OPT_JACOBI_SPLIT] == 0;
}

extern "C" int ishmemx_jacobi(double *buf0, double *buf1, uint64_t *sig, size_t ny, size_t nx, int iters,
                              int overlap, int groups_per_pe, int threads, double *residual_sq_host)
{
    ISHMEMI_REQUIRE_INIT();
    auto &g = g_ishmem;
    bool by_columns = false;
    int rc = jacobi_check(buf0, buf1, sig, ny, nx, iters, &groups_per_pe, threads, &by_columns);
    if (rc) return rc;
    if (jacobi_per_sweep(threads, nx)) {
        jacobi_plan pl;
        /* a launch of k > 2 sweeps parks its third to k-th halo rows in 2 (k - 2) extra symmetric rows;
         * without room for them in the heap the call falls back to shallower launches */
        double *xh = nullptr;
        for (int kmax : {JW_MAX_DEPTH, 4, 2}) {
            jacobi_make_plan(ny, nx, iters, kmax, &pl);
            if (pl.xh_side == 0) break;
            xh = (double *)ishmem_malloc(2 * (size_t)pl.xh_side * nx * sizeof(double));
            if (xh) break;
        }
        double *partial = nullptr;
        if (residual_sq_host)
            rc = ishmemi_cuda(cudaMalloc((void **)&partial, (pl.blocks_last ? pl.blocks_last : 1) * 8), "cudaMalloc");
        if (!rc) rc = jacobi_launch_sweeps(buf0, buf1, sig, ny, nx, iters, overlap, pl, partial, xh);
        if (!rc && residual_sq_host) {
            double sum = 0.0;
            if (pl.blocks_last) {
                std::vector<double> part(pl.blocks_last);
                rc = ishmemi_cuda(cudaMemcpy(part.data(), partial, pl.blocks_last * 8, cudaMemcpyDeviceToHost), "cudaMemcpy");
                for (size_t i = 0; i < pl.blocks_last; ++i) sum += part[i];
            }
            *residual_sq_host = sum;
        }
        cudaFree(partial);
        if (xh) ishmem_free(xh);
        return rc;
    }
    const size_t nblocks = (size_t)g.npes * groups_per_pe;
    /* scratch: per-block sweep counters and residual partials */
    char *scratch = nullptr;
    ISHMEMI_CUDA(cudaMalloc((void **)&scratch, nblocks * 16));
    jacobi_args a;
    rc = jacobi_launch(buf0, buf1, sig, ny, nx, iters, overlap, groups_per_pe, threads, by_columns, scratch, &a);
    if (!rc && residual_sq_host) {
        std::vector<double> part(nblocks);
        rc = ishmemi_cuda(cudaMemcpy(part.data(), a.partial, nblocks * 8, cudaMemcpyDeviceToHost), "cudaMemcpy");
        double sum = 0.0;
        for (size_t i = 0; i < nblocks; ++i) sum += part[i];
        *residual_sq_host = sum;
    }
    cudaFree(scratch);
    return rc;
}

/* ---- Jacobi without any allocation ---------------------------------------------------------
 * Some callers may not allocate device memory when they call into the library: code running
 * while a memory pool is frozen, inside a latency-critical loop where cudaMalloc's implicit
 * device synchronisation is unacceptable, or under an allocator that owns the whole device.
 * For them the per-block sweep counters and residual partials of the Jacobi kernel live in this
 * fixed array instead of a cudaMalloc'ed buffer.  Every GPU that loads the library holds these
 * 32 KiB until the process exits. */
#define ISHMEMX_JACOBI_NOALLOC_MAX_BLOCKS 2048
static __device__ __align__(256) unsigned char g_jacobi_scratch[ISHMEMX_JACOBI_NOALLOC_MAX_BLOCKS * 16];

/* device address of g_jacobi_scratch per device ordinal, resolved on first use: in host code the
 * symbol's name is only a handle, never a pointer a kernel may dereference */
static void *g_jacobi_scratch_addr[64] = {};

static int jacobi_scratch_for_current_device(void **out)
{
    int dev = 0;
    ISHMEMI_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return ISHMEM_ERR_ARG;
    if (!g_jacobi_scratch_addr[dev]) {
        void *p = nullptr;
        ISHMEMI_CUDA(cudaGetSymbolAddress(&p, g_jacobi_scratch));
        g_jacobi_scratch_addr[dev] = p;
    }
    *out = g_jacobi_scratch_addr[dev];
    return ISHMEM_OK;
}

extern "C" int ishmemx_jacobi_noalloc(double *buf0, double *buf1, uint64_t *sig, size_t ny, size_t nx, int iters,
                                      int overlap, int groups_per_pe, int threads, double *residual_sq_host)
{
    ISHMEMI_REQUIRE_INIT();
    auto &g = g_ishmem;
    bool by_columns = false;
    int rc = jacobi_check(buf0, buf1, sig, ny, nx, iters, &groups_per_pe, threads, &by_columns);
    if (rc == ISHMEM_ERR_ARG) return rc;
    const size_t nblocks = (size_t)g.npes * groups_per_pe;
    if (nblocks > ISHMEMX_JACOBI_NOALLOC_MAX_BLOCKS) {
        g.last_cuda_error = "ishmemx_jacobi_noalloc: npes * groups_per_pe exceeds the fixed scratch (2048 blocks)";
        return ISHMEM_ERR_ARG;
    }
    if (rc) return rc;
    void *scratch = nullptr;
    if ((rc = jacobi_scratch_for_current_device(&scratch))) return rc;
    /* the array keeps the previous call's counters; jacobi_launch clears the part this call uses */
    jacobi_args a;
    rc = jacobi_launch(buf0, buf1, sig, ny, nx, iters, overlap, groups_per_pe, threads, by_columns, scratch, &a);
    if (!rc && residual_sq_host) {
        double part[ISHMEMX_JACOBI_NOALLOC_MAX_BLOCKS];
        rc = ishmemi_cuda(cudaMemcpy(part, a.partial, nblocks * 8, cudaMemcpyDeviceToHost), "cudaMemcpy");
        double sum = 0.0;
        for (size_t i = 0; i < nblocks; ++i) sum += part[i];
        *residual_sq_host = sum;
    }
    return rc;
}
