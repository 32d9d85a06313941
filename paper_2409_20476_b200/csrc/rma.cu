/* Host entry points and launch kernels for RMA, signalling and point-to-point waits.
 * The kernels only slice the message and call the device API of ishmem_device.cuh: all
 * data movement happens in the library's device routines. */
#include "internal.h"

struct rma_args {
    char *dest;        /* single-PE launch: local to my_pe (or private); SPMD: PE 0's copy */
    const char *src;
    size_t nbytes;
    int my_pe;         /* >= 0: single-PE launch; -1: SPMD over all PEs */
    int pe;            /* target PE, or the shift for SPMD */
    int is_get;
    int groups;        /* blocks per PE */
    unsigned staging_bytes;
    /* optional signal (single-PE put only) */
    unsigned long long *sig;
    unsigned long long sig_value;
    int sig_op;
    int has_sig;
};

/* Slice [begin, begin+len) of an n-byte message for collaboration unit `u` of `units`:
 * equal slices rounded up to a multiple of 128 bytes, so every slice keeps the alignment
 * of the message start. */
__device__ __forceinline__ void slice_of(size_t n, unsigned long long u, unsigned long long units,
                                         size_t *begin, size_t *len)
{
    size_t per = (size_t)((n + units - 1) / units);
    per = (per + 127) & ~(size_t)127;
    size_t b = per * u;
    if (b >= n) {
        *begin = n;
        *len = 0;
    } else {
        *begin = b;
        *len = (n - b < per) ? (n - b) : per;
    }
}

template <int LEVEL>
__global__ void __launch_bounds__(1024) k_rma(const ishmem_ctx_t *ctxs, rma_args a)
{
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    int my, g;
    if (a.my_pe < 0) {
        const int npes = ctxs[0].npes;
        my = (int)(blockIdx.x % (unsigned)npes); /* consecutive blocks belong to different PEs */
        g = (int)(blockIdx.x / (unsigned)npes);
    } else {
        my = a.my_pe;
        g = (int)blockIdx.x;
    }
    const ishmem_ctx_t *ctx = ctxs + my;
    char *dest = a.dest;
    const char *src = a.src;
    int target = a.pe;
    if (a.my_pe < 0) {
        const long long off = ctx->heap_base - ctxs[0].heap_base;
        dest += off;
        src += off;
        target = (my + a.pe) % ctx->npes;
    }
    size_t begin, len;
    if (LEVEL == ISHMEMX_WORK_ITEM) {
        slice_of(a.nbytes, (unsigned long long)g * blockDim.x + threadIdx.x,
                 (unsigned long long)a.groups * blockDim.x, &begin, &len);
        if (len) {
            if (a.is_get) ishmem_getmem(ctx, dest + begin, src + begin, len, target);
            else ishmem_putmem(ctx, dest + begin, src + begin, len, target);
        }
    } else if (LEVEL == ISHMEMX_SUB_GROUP) {
        const unsigned wpb = blockDim.x >> 5;
        slice_of(a.nbytes, (unsigned long long)g * wpb + (threadIdx.x >> 5),
                 (unsigned long long)a.groups * wpb, &begin, &len);
        if (a.is_get) ishmemx_getmem_sub_group(ctx, dest + begin, src + begin, len, target);
        else ishmemx_putmem_sub_group(ctx, dest + begin, src + begin, len, target);
    } else if (LEVEL == ISHMEMX_WORK_GROUP_ENGINE) {
        slice_of(a.nbytes, (unsigned long long)g, (unsigned long long)a.groups, &begin, &len);
        /* non-blocking request, then quiet: exercises the per-PE completion counter */
        if (a.is_get) ishmemx_getmem_engine_work_group(ctx, dest + begin, src + begin, len, target, false);
        else ishmemx_putmem_engine_work_group(ctx, dest + begin, src + begin, len, target, false);
        ishmemx_quiet_work_group(ctx);
    } else {
        ishmemx_staging_t st = {nullptr, 0};
        if (LEVEL == ISHMEMX_WORK_GROUP_BULK) {
            st.smem = dyn_smem;
            st.bytes = a.staging_bytes;
        }
        slice_of(a.nbytes, (unsigned long long)g, (unsigned long long)a.groups, &begin, &len);
        if (a.is_get) ishmemx_getmem_work_group(ctx, dest + begin, src + begin, len, target, st);
        else ishmemx_putmem_work_group(ctx, dest + begin, src + begin, len, target, st);
    }
    if (a.has_sig) {
        /* host-initiated put_signal runs as one block: after the block barrier its leader
         * releases the signal */
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long *rs = ishmem_ptr(ctx, a.sig, target);
            if (rs) ishmemi::signal_update(rs, a.sig_value, a.sig_op); /* release: cumulative over the block */
        }
    }
}

/* scalar p: one thread stores one element */
template <typename T>
__global__ void k_p(const ishmem_ctx_t *ctxs, int my_pe, T *dest_local, T value, int pe)
{
    ishmem_p<T>(ctxs + my_pe, dest_local, value, pe);
}
template <typename T>
__global__ void k_g(const ishmem_ctx_t *ctxs, int my_pe, T *out_host_mapped, const T *src_local, int pe)
{
    *out_host_mapped = ishmem_g<T>(ctxs + my_pe, src_local, pe);
}

__global__ void k_wait_until(const ishmem_ctx_t *ctxs, int my_pe, const unsigned long long *ivar,
                             int cmp, unsigned long long value)
{
    ishmem_uint64_wait_until(ctxs + my_pe, ivar, cmp, value);
}

/* strided put/get: every block takes tiles of K_STRIDED_TILE consecutive elements (its threads share a
 * tile: neighbouring threads take neighbouring elements, four per thread in flight); blocks start in
 * index order, so the running blocks sweep one window of the source and of the destination together,
 * as in the contiguous copies.  The grid covers the message with one tile per block up to the launch
 * limit, beyond which a block moves on by the grid's width. */
#define K_STRIDED_TILE 1024u
__global__ void __launch_bounds__(256) k_strided(const ishmem_ctx_t *ctxs, int my_pe, char *dest, const char *src,
                                                 size_t dst, size_t sst, size_t nelems, unsigned es, int pe, int is_get)
{
    const ishmem_ctx_t *ctx = ctxs + my_pe;
    char *d = dest;
    const char *s = src;
    if (is_get) s = ishmem_ptr(ctx, src, pe);
    else d = ishmem_ptr(ctx, dest, pe);
    if (!d || !s) return;
    for (size_t lo = (size_t)blockIdx.x * K_STRIDED_TILE; lo < nelems; lo += (size_t)gridDim.x * K_STRIDED_TILE) {
        const size_t n = nelems - lo < K_STRIDED_TILE ? nelems - lo : K_STRIDED_TILE;
        ishmemi::strided_copy_any(d + lo * dst * es, s + lo * sst * es, dst, sst, n, es, threadIdx.x, blockDim.x);
    }
}

/* which: 0 all, 1 any, 2 some; results (index / count + indices) go to host-mapped memory */
__global__ void k_wait_many(const ishmem_ctx_t *ctxs, int my_pe, const unsigned long long *ivars, size_t nelems,
                            int cmp, unsigned long long value, int which, unsigned long long *out, const int *status)
{
    const ishmem_ctx_t *ctx = ctxs + my_pe;
    if (which == 0) {
        ishmem_uint64_wait_until_all(ctx, ivars, nelems, cmp, value, status);
    } else if (which == 1) {
        size_t idx = 0;
        int rc = ishmem_uint64_wait_until_any(ctx, ivars, nelems, cmp, value, &idx, status);
        out[0] = (unsigned long long)(long long)rc;
        out[1] = idx;
    } else {
        size_t cnt = 0;
        int rc = ishmem_uint64_wait_until_some(ctx, ivars, nelems, (size_t *)(out + 2), cmp, value, &cnt, status);
        out[0] = (unsigned long long)(long long)rc;
        out[1] = cnt;
    }
}

__global__ void k_test(const ishmem_ctx_t *ctxs, int my_pe, const unsigned long long *ivar, int cmp,
                       unsigned long long value, int *out)
{
    *out = ishmem_uint64_test(ctxs + my_pe, ivar, cmp, value);
}

/* ---- launch helpers --------------------------------------------------------------------- */

static unsigned g_bulk_smem = 0; /* the size the kernel's attribute was last set for */

static unsigned bulk_staging_bytes()
{
    /* ring of shared-memory stages: one block per SM with a deep ring measured best on B200
     * (ISHMEMX_OPT_BULK_SMEM holds the size) */
    unsigned want = (unsigned)g_ishmem.opt[ISHMEMX_OPT_BULK_SMEM];
    if (want > g_ishmem.max_dyn_smem) want = (unsigned)g_ishmem.max_dyn_smem;
    if (g_bulk_smem != want) {
        cudaFuncSetAttribute(k_rma<ISHMEMX_WORK_GROUP_BULK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)want);
        g_bulk_smem = want;
    }
    return g_bulk_smem;
}

static int launch_rma(cudaStream_t s, rma_args a, int level, int threads, unsigned blocks)
{
    if (threads < 1 || threads > 1024 || blocks == 0) return ISHMEM_ERR_ARG;
    if (level == ISHMEMX_SUB_GROUP && (threads % 32)) return ISHMEM_ERR_ARG;
    const ishmem_ctx_t *ctxs = g_ishmem.d_ctx;
    switch (level) {
    case ISHMEMX_WORK_ITEM: k_rma<ISHMEMX_WORK_ITEM><<<blocks, threads, 0, s>>>(ctxs, a); break;
    case ISHMEMX_SUB_GROUP: k_rma<ISHMEMX_SUB_GROUP><<<blocks, threads, 0, s>>>(ctxs, a); break;
    case ISHMEMX_WORK_GROUP: k_rma<ISHMEMX_WORK_GROUP><<<blocks, threads, 0, s>>>(ctxs, a); break;
    case ISHMEMX_WORK_GROUP_BULK:
        a.staging_bytes = bulk_staging_bytes();
        k_rma<ISHMEMX_WORK_GROUP_BULK><<<blocks, threads, a.staging_bytes, s>>>(ctxs, a);
        break;
    case ISHMEMX_WORK_GROUP_ENGINE:
        if (g_ishmem.h_ctx[0].proxy == nullptr) return ISHMEM_ERR_ARG; /* no host proxy running */
        k_rma<ISHMEMX_WORK_GROUP_ENGINE><<<blocks, threads, 0, s>>>(ctxs, a);
        /* This kernel waits for the host proxy, and the proxy's copy needs a free hardware queue:
         * work enqueued behind the kernel can end up in front of that copy (streams share the
         * queues), which would stall both until the wait gives up.  So the call returns only when
         * the kernel has finished -- nothing can be queued behind it. */
        ishmemi_count_launch();
        {
            int rc = ishmemi_check_launch("k_rma");
            if (rc) return rc;
        }
        return ishmemi_cuda(cudaStreamSynchronize(s), "cudaStreamSynchronize(engine level)");
    default: return ISHMEM_ERR_ARG;
    }
    ishmemi_count_launch();
    int rc = ishmemi_check_launch("k_rma");
    /* a work-group slice at or above the device-side cutover goes to the proxy as well: same rule */
    const bool may_wait_for_proxy = (level == ISHMEMX_WORK_GROUP || level == ISHMEMX_WORK_GROUP_BULK) &&
                                    g_ishmem.h_ctx[0].proxy != nullptr && g_ishmem.wg_cutover != (size_t)-1 &&
                                    a.nbytes >= g_ishmem.wg_cutover;
    if (!rc && may_wait_for_proxy) rc = ishmemi_cuda(cudaStreamSynchronize(s), "cudaStreamSynchronize(cutover)");
    return rc;
}

/* Validates one RMA request and resolves addresses: the symmetric side must lie in the heap;
 * the other side is my_pe's copy if symmetric, else taken as a private device pointer. */
static int resolve(int my_pe, void *dest, const void *src, size_t n, int pe, bool is_get,
                   char **dest_local, const char **src_local)
{
    ISHMEMI_REQUIRE_INIT();
    if (ishmemi_check_pe(my_pe) || ishmemi_check_pe(pe)) return ISHMEM_ERR_INVALID_PE;
    if (n && (!dest || !src)) return ISHMEM_ERR_ARG;
    const void *sym = is_get ? src : (const void *)dest;
    if (ishmemi_sym_offset(sym, n) < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    *dest_local = ishmemi_localise(dest, n, my_pe);
    *src_local = ishmemi_localise(src, n, my_pe);
    return ISHMEM_OK;
}

/* geometry of a host-initiated transfer that the caller did not shape */
static void auto_geometry(size_t n, int *threads, unsigned *blocks, int *level)
{
    if (n <= 1024) {
        *threads = 64;
        *blocks = 1;
        *level = ISHMEMX_WORK_GROUP;
    } else if (n <= (256u << 10)) {
        *threads = 256;
        *blocks = (unsigned)((n + 16383) / 16384);
        *level = ISHMEMX_WORK_GROUP;
    } else {
        /* one tile (32 KiB for large messages) per block.  Blocks start in index order, so the running blocks sweep one
         * short window of the source and of the destination; measured on B200 that moves more
         * bytes per second (6.8 TB/s at 256 MiB per PE) than a resident grid streaming long slices,
         * by loads and stores or through the TMA ring (6.4) */
        *threads = 256;
        /* 128 bytes per thread when that still gives every SM four blocks, down to 16 for messages
         * of a few MiB, which need the parallelism more than the long bursts */
        size_t per_thread = 128;
        while (per_thread > 16 && n / (256 * per_thread) < (size_t)g_ishmem.sm_count * 4) per_thread >>= 1;
        const size_t tile = 256 * per_thread, b = (n + tile - 1) / tile;
        *blocks = (unsigned)(b < 0x7fffffffu ? b : 0x7fffffffu);
        *level = ISHMEMX_WORK_GROUP;
    }
}

static int rma_common(int my_pe, void *dest, const void *src, size_t n, int pe, bool is_get, bool nbi)
{
    char *dl;
    const char *sl;
    int rc = resolve(my_pe, dest, src, n, pe, is_get, &dl, &sl);
    if (rc) return rc;
    if (n == 0) return ISHMEM_OK;
    auto &g = g_ishmem;
    if (n >= g.cutover[0] && n < g.cutover_put_upto) {
        /* copy-engine path: translate the remote side on the host */
        char *d = is_get ? dl : dl + ((long long)pe - my_pe) * (long long)g.heap_bytes;
        const char *s = is_get ? sl + ((long long)pe - my_pe) * (long long)g.heap_bytes : sl;
        return ishmemi_engine_copy(my_pe, d, s, n, !nbi);
    }
    rma_args a = {};
    a.dest = dl;
    a.src = sl;
    a.nbytes = n;
    a.my_pe = my_pe;
    a.pe = pe;
    a.is_get = is_get;
    int threads, level;
    unsigned blocks;
    auto_geometry(n, &threads, &blocks, &level);
    a.groups = (int)blocks;
    return launch_rma(ishmemi_pe_stream_for_op(my_pe), a, level, threads, blocks);
}

extern "C" int ishmem_putmem(int my_pe, void *dest, const void *src, size_t nbytes, int pe)
{
    return rma_common(my_pe, dest, src, nbytes, pe, false, false);
}
extern "C" int ishmem_getmem(int my_pe, void *dest, const void *src, size_t nbytes, int pe)
{
    return rma_common(my_pe, dest, src, nbytes, pe, true, false);
}
extern "C" int ishmem_putmem_nbi(int my_pe, void *dest, const void *src, size_t nbytes, int pe)
{
    return rma_common(my_pe, dest, src, nbytes, pe, false, true);
}
extern "C" int ishmem_getmem_nbi(int my_pe, void *dest, const void *src, size_t nbytes, int pe)
{
    return rma_common(my_pe, dest, src, nbytes, pe, true, true);
}

template <typename T>
static int typed_rma(int my_pe, T *dest, const T *src, size_t nelems, int pe, bool is_get, bool nbi)
{
    if (((uintptr_t)dest | (uintptr_t)src) % sizeof(T)) return ISHMEM_ERR_ALIGN;
    if (nelems > (size_t)-1 / sizeof(T)) return ISHMEM_ERR_ARG;
    return rma_common(my_pe, dest, src, nelems * sizeof(T), pe, is_get, nbi);
}

template <typename T>
static int typed_p(int my_pe, T *dest, T value, int pe)
{
    ISHMEMI_REQUIRE_INIT();
    if (ishmemi_check_pe(my_pe) || ishmemi_check_pe(pe)) return ISHMEM_ERR_INVALID_PE;
    if ((uintptr_t)dest % sizeof(T)) return ISHMEM_ERR_ALIGN;
    if (ishmemi_sym_offset(dest, sizeof(T)) < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    T *dl = (T *)ishmemi_localise(dest, sizeof(T), my_pe);
    k_p<T><<<1, 1, 0, ishmemi_pe_stream_for_op(my_pe)>>>(g_ishmem.d_ctx, my_pe, dl, value, pe);
    ishmemi_count_launch();
    return ishmemi_check_launch("k_p");
}

template <typename T>
static int typed_g(int my_pe, T *value_out_host, const T *src, int pe)
{
    ISHMEMI_REQUIRE_INIT();
    if (ishmemi_check_pe(my_pe) || ishmemi_check_pe(pe)) return ISHMEM_ERR_INVALID_PE;
    if (!value_out_host) return ISHMEM_ERR_ARG;
    if ((uintptr_t)src % sizeof(T)) return ISHMEM_ERR_ALIGN;
    if (ishmemi_sym_offset(src, sizeof(T)) < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    const T *sl = (const T *)ishmemi_localise(src, sizeof(T), my_pe);
    cudaStream_t s = ishmemi_pe_stream_for_op(my_pe);
    k_g<T><<<1, 1, 0, s>>>(g_ishmem.d_ctx, my_pe, (T *)g_ishmem.h_pinned, sl, pe);
    ishmemi_count_launch();
    int rc = ishmemi_check_launch("k_g");
    if (rc) return rc;
    ISHMEMI_CUDA(cudaStreamSynchronize(s));
    *value_out_host = *(T *)g_ishmem.h_pinned;
    return ISHMEM_OK;
}

#define ISHMEMI_DEF_RMA(NAME, T)                                                                   \
    extern "C" int ishmem_##NAME##_put(int my_pe, T *dest, const T *src, size_t nelems, int pe)    \
    {                                                                                              \
        return typed_rma<T>(my_pe, dest, src, nelems, pe, false, false);                           \
    }                                                                                              \
    extern "C" int ishmem_##NAME##_get(int my_pe, T *dest, const T *src, size_t nelems, int pe)    \
    {                                                                                              \
        return typed_rma<T>(my_pe, dest, src, nelems, pe, true, false);                            \
    }                                                                                              \
    extern "C" int ishmem_##NAME##_put_nbi(int my_pe, T *dest, const T *src, size_t nelems, int pe) \
    {                                                                                              \
        return typed_rma<T>(my_pe, dest, src, nelems, pe, false, true);                            \
    }                                                                                              \
    extern "C" int ishmem_##NAME##_get_nbi(int my_pe, T *dest, const T *src, size_t nelems, int pe) \
    {                                                                                              \
        return typed_rma<T>(my_pe, dest, src, nelems, pe, true, true);                             \
    }                                                                                              \
    extern "C" int ishmem_##NAME##_p(int my_pe, T *dest, T value, int pe)                          \
    {                                                                                              \
        return typed_p<T>(my_pe, dest, value, pe);                                                 \
    }                                                                                              \
    extern "C" int ishmem_##NAME##_g(int my_pe, T *value_out_host, const T *src, int pe)           \
    {                                                                                              \
        return typed_g<T>(my_pe, value_out_host, src, pe);                                         \
    }
ISHMEMI_DEF_RMA(float, float)
ISHMEMI_DEF_RMA(double, double)
ISHMEMI_DEF_RMA(int, int)
ISHMEMI_DEF_RMA(long, long)
ISHMEMI_DEF_RMA(int32, int32_t)
ISHMEMI_DEF_RMA(int64, int64_t)
ISHMEMI_DEF_RMA(uint8, uint8_t)
ISHMEMI_DEF_RMA(uint32, uint32_t)
ISHMEMI_DEF_RMA(uint64, uint64_t)

static int strided(int my_pe, void *dest, const void *src, size_t dst, size_t sst, size_t nelems, size_t es, int pe,
                   bool is_get)
{
    ISHMEMI_REQUIRE_INIT();
    if (ishmemi_check_pe(my_pe) || ishmemi_check_pe(pe)) return ISHMEM_ERR_INVALID_PE;
    if (es != 1 && es != 2 && es != 4 && es != 8 && es != 16) return ISHMEM_ERR_ARG;
    if (dst < 1 || sst < 1) return ISHMEM_ERR_ARG;
    if (nelems == 0) return ISHMEM_OK;
    if (!dest || !src) return ISHMEM_ERR_ARG;
    if (((uintptr_t)dest | (uintptr_t)src) % es) return ISHMEM_ERR_ALIGN;
    if ((nelems - 1) > ((size_t)-1 / es - 1) / (dst > sst ? dst : sst)) return ISHMEM_ERR_ARG;
    const size_t dspan = ((nelems - 1) * dst + 1) * es, sspan = ((nelems - 1) * sst + 1) * es;
    if (ishmemi_sym_offset(is_get ? src : (const void *)dest, is_get ? sspan : dspan) < 0)
        return ISHMEM_ERR_NOT_SYMMETRIC;
    /* both strides 1: a contiguous message, which the vectorised put / get moves at twice the rate of
     * element-sized accesses */
    if (dst == 1 && sst == 1) return rma_common(my_pe, dest, src, nelems * es, pe, is_get, false);
    char *dl = ishmemi_localise(dest, dspan, my_pe);
    const char *sl = ishmemi_localise(src, sspan, my_pe);
    size_t blocks = (nelems + K_STRIDED_TILE - 1) / K_STRIDED_TILE;
    if (blocks > 0x7fffffffu) blocks = 0x7fffffffu;
    k_strided<<<(unsigned)blocks, 256, 0, ishmemi_pe_stream_for_op(my_pe)>>>(g_ishmem.d_ctx, my_pe, dl, sl, dst, sst,
                                                                             nelems, (unsigned)es, pe, is_get ? 1 : 0);
    ishmemi_count_launch();
    return ishmemi_check_launch("k_strided");
}
extern "C" int ishmemx_iputmem(int my_pe, void *dest, const void *src, size_t dst, size_t sst, size_t nelems,
                               size_t elem_size, int pe)
{
    return strided(my_pe, dest, src, dst, sst, nelems, elem_size, pe, false);
}
extern "C" int ishmemx_igetmem(int my_pe, void *dest, const void *src, size_t dst, size_t sst, size_t nelems,
                               size_t elem_size, int pe)
{
    return strided(my_pe, dest, src, dst, sst, nelems, elem_size, pe, true);
}
#define ISHMEMI_DEF_STRIDED(NAME, T)                                                                          \
    extern "C" int ishmem_##NAME##_iput(int my_pe, T *dest, const T *src, size_t dst, size_t sst, size_t nelems, \
                                        int pe)                                                               \
    {                                                                                                         \
        return strided(my_pe, dest, src, dst, sst, nelems, sizeof(T), pe, false);                             \
    }                                                                                                         \
    extern "C" int ishmem_##NAME##_iget(int my_pe, T *dest, const T *src, size_t dst, size_t sst, size_t nelems, \
                                        int pe)                                                               \
    {                                                                                                         \
        return strided(my_pe, dest, src, dst, sst, nelems, sizeof(T), pe, true);                              \
    }
ISHMEMI_DEF_STRIDED(float, float)
ISHMEMI_DEF_STRIDED(double, double)
ISHMEMI_DEF_STRIDED(int, int)
ISHMEMI_DEF_STRIDED(long, long)
ISHMEMI_DEF_STRIDED(int32, int32_t)
ISHMEMI_DEF_STRIDED(int64, int64_t)
ISHMEMI_DEF_STRIDED(uint8, uint8_t)
ISHMEMI_DEF_STRIDED(uint32, uint32_t)
ISHMEMI_DEF_STRIDED(uint64, uint64_t)

static int on_device(int my_pe, void *dest, const void *src, size_t n, int pe, int level, int threads,
                     int groups, bool is_get)
{
    char *dl;
    const char *sl;
    int rc = resolve(my_pe, dest, src, n, pe, is_get, &dl, &sl);
    if (rc) return rc;
    if (groups < 1) return ISHMEM_ERR_ARG;
    rma_args a = {};
    a.dest = dl;
    a.src = sl;
    a.nbytes = n;
    a.my_pe = my_pe;
    a.pe = pe;
    a.is_get = is_get;
    a.groups = groups;
    return launch_rma(ishmemi_pe_stream_for_op(my_pe), a, level, threads, (unsigned)groups);
}

extern "C" int ishmemx_putmem_on_device(int my_pe, void *dest, const void *src, size_t nbytes, int pe,
                                        int level, int threads, int groups)
{
    return on_device(my_pe, dest, src, nbytes, pe, level, threads, groups, false);
}
extern "C" int ishmemx_getmem_on_device(int my_pe, void *dest, const void *src, size_t nbytes, int pe,
                                        int level, int threads, int groups)
{
    return on_device(my_pe, dest, src, nbytes, pe, level, threads, groups, true);
}

static int engine_rma(int my_pe, void *dest, const void *src, size_t n, int pe, bool is_get)
{
    char *dl;
    const char *sl;
    int rc = resolve(my_pe, dest, src, n, pe, is_get, &dl, &sl);
    if (rc) return rc;
    if (n == 0) return ISHMEM_OK;
    const long long shift = ((long long)pe - my_pe) * (long long)g_ishmem.heap_bytes;
    return ishmemi_engine_copy(my_pe, is_get ? dl : dl + shift, is_get ? sl + shift : sl, n, true);
}
extern "C" int ishmemx_putmem_copy_engine(int my_pe, void *dest, const void *src, size_t nbytes, int pe)
{
    return engine_rma(my_pe, dest, src, nbytes, pe, false);
}
extern "C" int ishmemx_getmem_copy_engine(int my_pe, void *dest, const void *src, size_t nbytes, int pe)
{
    return engine_rma(my_pe, dest, src, nbytes, pe, true);
}

/* groups == 0 in a caller-shaped launch: one tile of 128 bytes per thread for every block */
static int tile_groups(size_t n, int threads, int launches_sharing_grid)
{
    const size_t tile = (size_t)threads * 128, want = (n + tile - 1) / tile;
    const size_t most = 0x7fffffffu / (size_t)launches_sharing_grid;
    return (int)(want < 1 ? 1 : (want < most ? want : most));
}

static int spmd(void *dest, const void *src, size_t n, int shift, int level, int threads, int groups,
                bool is_get)
{
    ISHMEMI_REQUIRE_INIT();
    auto &g = g_ishmem;
    if (groups < 0 || shift < 0 || threads < 1) return ISHMEM_ERR_ARG;
    if (ishmemi_sym_offset(dest, n) < 0 || ishmemi_sym_offset(src, n) < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    if (groups == 0) groups = tile_groups(n, threads, g.npes);
    rma_args a = {};
    a.dest = (char *)dest;
    a.src = (const char *)src;
    a.nbytes = n;
    a.my_pe = -1;
    a.pe = shift % g.npes;
    a.is_get = is_get;
    a.groups = groups;
    cudaStream_t s;
    int rc = ishmemi_team_stream_begin(ISHMEM_TEAM_WORLD, &s);
    if (rc) return rc;
    rc = launch_rma(s, a, level, threads, (unsigned)groups * (unsigned)g.npes);
    ishmemi_team_stream_end();
    return rc;
}
extern "C" int ishmemx_putmem_spmd(void *dest, const void *src, size_t nbytes, int shift, int level,
                                   int threads, int groups)
{
    return spmd(dest, src, nbytes, shift, level, threads, groups, false);
}
extern "C" int ishmemx_getmem_spmd(void *dest, const void *src, size_t nbytes, int shift, int level,
                                   int threads, int groups)
{
    return spmd(dest, src, nbytes, shift, level, threads, groups, true);
}

extern "C" int ishmemx_putmem_spmd_copy_engine(void *dest, const void *src, size_t nbytes, int shift)
{
    ISHMEMI_REQUIRE_INIT();
    auto &g = g_ishmem;
    long long doff = ishmemi_sym_offset(dest, nbytes), soff = ishmemi_sym_offset(src, nbytes);
    if (doff < 0 || soff < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    if (shift < 0) return ISHMEM_ERR_ARG;
    cudaStream_t s;
    int rc = ishmemi_team_stream_begin(ISHMEM_TEAM_WORLD, &s);
    if (rc) return rc;
    for (int p = 0; p < g.npes && !rc; ++p) {
        int t = (p + shift) % g.npes;
        rc = ishmemi_cuda(cudaMemcpyAsync(g.base + (size_t)t * g.heap_bytes + doff,
                                          g.base + (size_t)p * g.heap_bytes + soff, nbytes,
                                          cudaMemcpyDeviceToDevice, s),
                          "cudaMemcpyAsync");
    }
    ishmemi_team_stream_end();
    return rc;
}

/* ---- signalling, waits, ordering -------------------------------------------------------- */

extern "C" int ishmem_putmem_signal(int my_pe, void *dest, const void *src, size_t nbytes,
                                    uint64_t *sig_addr, uint64_t signal, int sig_op, int pe)
{
    char *dl;
    const char *sl;
    int rc = resolve(my_pe, dest, src, nbytes, pe, false, &dl, &sl);
    if (rc) return rc;
    if ((uintptr_t)sig_addr % 8) return ISHMEM_ERR_ALIGN;
    if (ishmemi_sym_offset(sig_addr, 8) < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    if (sig_op != ISHMEM_SIGNAL_SET && sig_op != ISHMEM_SIGNAL_ADD) return ISHMEM_ERR_ARG;
    rma_args a = {};
    a.dest = dl;
    a.src = sl;
    a.nbytes = nbytes;
    a.my_pe = my_pe;
    a.pe = pe;
    a.groups = 1; /* one work-group: payload, block barrier, then the leader's release */
    a.sig = (unsigned long long *)ishmemi_localise(sig_addr, 8, my_pe);
    a.sig_value = signal;
    a.sig_op = sig_op;
    a.has_sig = 1;
    int threads = nbytes <= 4096 ? 128 : 1024;
    return launch_rma(ishmemi_pe_stream_for_op(my_pe), a, ISHMEMX_WORK_GROUP, threads, 1);
}

extern "C" int ishmem_uint64_wait_until(int my_pe, uint64_t *ivar, int cmp, uint64_t value)
{
    ISHMEMI_REQUIRE_INIT();
    if (ishmemi_check_pe(my_pe)) return ISHMEM_ERR_INVALID_PE;
    if ((uintptr_t)ivar % 8) return ISHMEM_ERR_ALIGN;
    if (ishmemi_sym_offset(ivar, 8) < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    if (cmp < ISHMEM_CMP_EQ || cmp > ISHMEM_CMP_LE) return ISHMEM_ERR_ARG;
    const unsigned long long *il = (const unsigned long long *)ishmemi_localise(ivar, 8, my_pe);
    k_wait_until<<<1, 1, 0, ishmemi_pe_stream_for_op(my_pe)>>>(g_ishmem.d_ctx, my_pe, il, cmp, value);
    ishmemi_count_launch();
    return ishmemi_check_launch("k_wait_until");
}

extern "C" int ishmem_uint64_test(int my_pe, uint64_t *ivar, int cmp, uint64_t value, int *result)
{
    ISHMEMI_REQUIRE_INIT();
    if (ishmemi_check_pe(my_pe)) return ISHMEM_ERR_INVALID_PE;
    if ((uintptr_t)ivar % 8) return ISHMEM_ERR_ALIGN;
    if (ishmemi_sym_offset(ivar, 8) < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    if (cmp < ISHMEM_CMP_EQ || cmp > ISHMEM_CMP_LE || !result) return ISHMEM_ERR_ARG;
    const unsigned long long *il = (const unsigned long long *)ishmemi_localise(ivar, 8, my_pe);
    cudaStream_t s = ishmemi_pe_stream_for_op(my_pe);
    k_test<<<1, 1, 0, s>>>(g_ishmem.d_ctx, my_pe, il, cmp, value, (int *)g_ishmem.h_pinned);
    ishmemi_count_launch();
    int rc = ishmemi_check_launch("k_test");
    if (rc) return rc;
    ISHMEMI_CUDA(cudaStreamSynchronize(s));
    *result = *(int *)g_ishmem.h_pinned;
    return ISHMEM_OK;
}

static int wait_many(int my_pe, uint64_t *ivars, size_t nelems, const int *status, int cmp, uint64_t value, int which,
                     size_t *index, size_t *indices, size_t *count)
{
    ISHMEMI_REQUIRE_INIT();
    if (ishmemi_check_pe(my_pe)) return ISHMEM_ERR_INVALID_PE;
    if ((uintptr_t)ivars % 8) return ISHMEM_ERR_ALIGN;
    if (nelems > 256) return ISHMEM_ERR_ARG;
    if (ishmemi_sym_offset(ivars, nelems * 8) < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    if (cmp < ISHMEM_CMP_EQ || cmp > ISHMEM_CMP_LE) return ISHMEM_ERR_ARG;
    if ((which == 1 && !index) || (which == 2 && (!indices || !count))) return ISHMEM_ERR_ARG;
    const unsigned long long *il = (const unsigned long long *)ishmemi_localise(ivars, nelems * 8, my_pe);
    cudaStream_t s = ishmemi_pe_stream_for_op(my_pe);
    unsigned long long *out = (unsigned long long *)g_ishmem.h_pinned; /* 4096 B: 2 + 256 words */
    k_wait_many<<<1, 1, 0, s>>>(g_ishmem.d_ctx, my_pe, il, nelems, cmp, value, which, out, status);
    ishmemi_count_launch();
    int rc = ishmemi_check_launch("k_wait_many");
    if (rc || which == 0) return rc;
    ISHMEMI_CUDA(cudaStreamSynchronize(s));
    if ((long long)out[0]) return (int)(long long)out[0];
    if (which == 1) {
        *index = (size_t)out[1];
    } else {
        *count = (size_t)out[1];
        for (size_t k = 0; k < *count; ++k) indices[k] = (size_t)out[2 + k];
    }
    return ISHMEM_OK;
}
extern "C" int ishmem_uint64_wait_until_all(int my_pe, uint64_t *ivars, size_t nelems, const int *status, int cmp,
                                            uint64_t value)
{
    return wait_many(my_pe, ivars, nelems, status, cmp, value, 0, nullptr, nullptr, nullptr);
}
extern "C" int ishmem_uint64_wait_until_any(int my_pe, uint64_t *ivars, size_t nelems, const int *status, int cmp,
                                            uint64_t value, size_t *index)
{
    return wait_many(my_pe, ivars, nelems, status, cmp, value, 1, index, nullptr, nullptr);
}
extern "C" int ishmem_uint64_wait_until_some(int my_pe, uint64_t *ivars, size_t nelems, size_t *indices,
                                             const int *status, int cmp, uint64_t value, size_t *count)
{
    return wait_many(my_pe, ivars, nelems, status, cmp, value, 2, nullptr, indices, count);
}

extern "C" int ishmem_fence(int my_pe)
{
    ISHMEMI_REQUIRE_INIT();
    return ishmemi_check_pe(my_pe) ? ISHMEM_ERR_INVALID_PE : ISHMEM_OK;
}

extern "C" int ishmem_quiet(int my_pe)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    if (ishmemi_check_pe(my_pe)) return ISHMEM_ERR_INVALID_PE;
    if (g.nbi_pending[my_pe]) {
        ISHMEMI_CUDA(cudaEventRecord(g.ev_engine[my_pe], g.engine_stream[my_pe]));
        ISHMEMI_CUDA(cudaStreamWaitEvent(g.pe_stream[my_pe], g.ev_engine[my_pe], 0));
        g.nbi_pending[my_pe] = false;
        g.pe_dirty[my_pe] = true;
    }
    return ISHMEM_OK;
}

/* ---- end-to-end helper with host buffers --------------------------------------------------- */

extern "C" int ishmemx_host_put_ring(void *dest_host, const void *src_host, void *dest, void *src,
                                     size_t nbytes, int shift, int level, int threads, int groups)
{
    ISHMEMI_REQUIRE_INIT();
    auto &g = g_ishmem;
    if (!dest_host || !src_host) return ISHMEM_ERR_ARG;
    if (groups < 0 || shift < 0 || threads < 1) return ISHMEM_ERR_ARG;
    if (groups == 0) groups = tile_groups(nbytes, threads, 1);
    long long doff = ishmemi_sym_offset(dest, nbytes), soff = ishmemi_sym_offset(src, nbytes);
    if (doff < 0 || soff < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    /* One pipeline per PE on that PE's stream: payload in, the PE's put, and the copy back of the
     * destination that put has just filled.  The pipelines of different PEs overlap, so the bus
     * carries host-to-device and device-to-host traffic at the same time. */
    int rc = ISHMEM_OK;
    for (int p = 0; p < g.npes && !rc; ++p) {
        const int t = (p + shift) % g.npes;
        cudaStream_t s = ishmemi_pe_stream_for_op(p);
        rc = ishmemi_cuda(cudaMemcpyAsync(g.base + (size_t)p * g.heap_bytes + (size_t)soff,
                                          (const char *)src_host + (size_t)p * nbytes, nbytes, cudaMemcpyHostToDevice, s),
                          "cudaMemcpyAsync(H2D)");
        if (rc) break;
        rma_args a = {};
        a.dest = g.base + (size_t)p * g.heap_bytes + (size_t)doff; /* my_pe's copy: translated to t in the kernel */
        a.src = g.base + (size_t)p * g.heap_bytes + (size_t)soff;
        a.nbytes = nbytes;
        a.my_pe = p;
        a.pe = t;
        a.groups = groups;
        if (nbytes) rc = launch_rma(s, a, level, threads, (unsigned)groups);
        if (rc) break;
        rc = ishmemi_cuda(cudaMemcpyAsync((char *)dest_host + (size_t)t * nbytes,
                                          g.base + (size_t)t * g.heap_bytes + (size_t)doff, nbytes, cudaMemcpyDeviceToHost, s),
                          "cudaMemcpyAsync(D2H)");
    }
    for (int p = 0; p < g.npes; ++p) {
        int rc2 = ishmemi_cuda(cudaStreamSynchronize(g.pe_stream[p]), "cudaStreamSynchronize");
        if (!rc) rc = rc2;
    }
    return rc;
}
