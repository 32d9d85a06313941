/* Remote atomic memory operations: host-initiated single operations and the device-initiated
 * batches (one operation per GPU thread).  All atomics go through the device API of
 * ishmem_device.cuh (address translation + .gpu-scope atomic). */
#include "internal.h"

enum { AMO_ADD, AMO_INC, AMO_SET, AMO_FETCH, AMO_FETCH_ADD, AMO_FETCH_INC, AMO_SWAP, AMO_CAS, AMO_FETCH_AND,
       AMO_FETCH_OR, AMO_FETCH_XOR, AMO_AND, AMO_OR, AMO_XOR };

template <typename T>
__global__ void k_amo(const ishmem_ctx_t *ctxs, int my_pe, int op, T *target_local, T value, T cond, int pe,
                      T *out_host_mapped)
{
    const ishmem_ctx_t *ctx = ctxs + my_pe;
    T old = T();
    switch (op) {
    case AMO_ADD: ishmem_atomic_add<T>(ctx, target_local, value, pe); break;
    case AMO_INC: ishmem_atomic_inc<T>(ctx, target_local, pe); break;
    case AMO_SET: ishmem_atomic_set<T>(ctx, target_local, value, pe); break;
    case AMO_AND: ishmem_atomic_and<T>(ctx, target_local, value, pe); break;
    case AMO_OR: ishmem_atomic_or<T>(ctx, target_local, value, pe); break;
    case AMO_XOR: ishmem_atomic_xor<T>(ctx, target_local, value, pe); break;
    case AMO_FETCH: old = ishmem_atomic_fetch<T>(ctx, target_local, pe); break;
    case AMO_FETCH_ADD: old = ishmem_atomic_fetch_add<T>(ctx, target_local, value, pe); break;
    case AMO_FETCH_INC: old = ishmem_atomic_fetch_inc<T>(ctx, target_local, pe); break;
    case AMO_SWAP: old = ishmem_atomic_swap<T>(ctx, target_local, value, pe); break;
    case AMO_CAS: old = ishmem_atomic_compare_swap<T>(ctx, target_local, cond, value, pe); break;
    case AMO_FETCH_AND: old = ishmem_atomic_fetch_and<T>(ctx, target_local, value, pe); break;
    case AMO_FETCH_OR: old = ishmem_atomic_fetch_or<T>(ctx, target_local, value, pe); break;
    default: old = ishmem_atomic_fetch_xor<T>(ctx, target_local, value, pe); break;
    }
    if (out_host_mapped) *out_host_mapped = old;
}

/* D = the device-side type with the same size as the ABI type T */
template <typename T, typename D>
static int host_amo(int my_pe, int op, T *fetched_host, const T *target, T value, T cond, int pe, bool fetching)
{
    ISHMEMI_REQUIRE_INIT();
    auto &g = g_ishmem;
    if (ishmemi_check_pe(my_pe) || ishmemi_check_pe(pe)) return ISHMEM_ERR_INVALID_PE;
    if ((uintptr_t)target % sizeof(T)) return ISHMEM_ERR_ALIGN;
    if (ishmemi_sym_offset(target, sizeof(T)) < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    if (fetching && !fetched_host) return ISHMEM_ERR_ARG;
    D *tl = (D *)ishmemi_localise(target, sizeof(T), my_pe);
    cudaStream_t s = ishmemi_pe_stream_for_op(my_pe);
    k_amo<D><<<1, 1, 0, s>>>(g.d_ctx, my_pe, op, tl, (D)value, (D)cond, pe, fetching ? (D *)g.h_pinned : nullptr);
    ishmemi_count_launch();
    int rc = ishmemi_check_launch("k_amo");
    if (rc || !fetching) return rc;
    ISHMEMI_CUDA(cudaStreamSynchronize(s));
    *fetched_host = (T)(*(D *)g.h_pinned);
    return ISHMEM_OK;
}

#define ISHMEMI_DEF_AMO(NAME, T, D)                                                                               \
    extern "C" int ishmem_##NAME##_atomic_add(int my_pe, T *target, T value, int pe)                              \
    {                                                                                                             \
        return host_amo<T, D>(my_pe, AMO_ADD, nullptr, target, value, 0, pe, false);                              \
    }                                                                                                             \
    extern "C" int ishmem_##NAME##_atomic_inc(int my_pe, T *target, int pe)                                       \
    {                                                                                                             \
        return host_amo<T, D>(my_pe, AMO_INC, nullptr, target, 0, 0, pe, false);                                  \
    }                                                                                                             \
    extern "C" int ishmem_##NAME##_atomic_set(int my_pe, T *target, T value, int pe)                              \
    {                                                                                                             \
        return host_amo<T, D>(my_pe, AMO_SET, nullptr, target, value, 0, pe, false);                              \
    }                                                                                                             \
    extern "C" int ishmem_##NAME##_atomic_and(int my_pe, T *target, T value, int pe)                              \
    {                                                                                                             \
        return host_amo<T, D>(my_pe, AMO_AND, nullptr, target, value, 0, pe, false);                              \
    }                                                                                                             \
    extern "C" int ishmem_##NAME##_atomic_or(int my_pe, T *target, T value, int pe)                               \
    {                                                                                                             \
        return host_amo<T, D>(my_pe, AMO_OR, nullptr, target, value, 0, pe, false);                               \
    }                                                                                                             \
    extern "C" int ishmem_##NAME##_atomic_xor(int my_pe, T *target, T value, int pe)                              \
    {                                                                                                             \
        return host_amo<T, D>(my_pe, AMO_XOR, nullptr, target, value, 0, pe, false);                              \
    }                                                                                                             \
    extern "C" int ishmem_##NAME##_atomic_fetch(int my_pe, T *fetched_host, const T *target, int pe)              \
    {                                                                                                             \
        return host_amo<T, D>(my_pe, AMO_FETCH, fetched_host, target, 0, 0, pe, true);                            \
    }                                                                                                             \
    extern "C" int ishmem_##NAME##_atomic_fetch_add(int my_pe, T *fetched_host, T *target, T value, int pe)       \
    {                                                                                                             \
        return host_amo<T, D>(my_pe, AMO_FETCH_ADD, fetched_host, target, value, 0, pe, true);                    \
    }                                                                                                             \
    extern "C" int ishmem_##NAME##_atomic_fetch_inc(int my_pe, T *fetched_host, T *target, int pe)                \
    {                                                                                                             \
        return host_amo<T, D>(my_pe, AMO_FETCH_INC, fetched_host, target, 0, 0, pe, true);                        \
    }                                                                                                             \
    extern "C" int ishmem_##NAME##_atomic_swap(int my_pe, T *fetched_host, T *target, T value, int pe)            \
    {                                                                                                             \
        return host_amo<T, D>(my_pe, AMO_SWAP, fetched_host, target, value, 0, pe, true);                         \
    }                                                                                                             \
    extern "C" int ishmem_##NAME##_atomic_compare_swap(int my_pe, T *fetched_host, T *target, T cond, T value,    \
                                                       int pe)                                                    \
    {                                                                                                             \
        return host_amo<T, D>(my_pe, AMO_CAS, fetched_host, target, value, cond, pe, true);                       \
    }                                                                                                             \
    extern "C" int ishmem_##NAME##_atomic_fetch_and(int my_pe, T *fetched_host, T *target, T value, int pe)       \
    {                                                                                                             \
        return host_amo<T, D>(my_pe, AMO_FETCH_AND, fetched_host, target, value, 0, pe, true);                    \
    }                                                                                                             \
    extern "C" int ishmem_##NAME##_atomic_fetch_or(int my_pe, T *fetched_host, T *target, T value, int pe)        \
    {                                                                                                             \
        return host_amo<T, D>(my_pe, AMO_FETCH_OR, fetched_host, target, value, 0, pe, true);                     \
    }                                                                                                             \
    extern "C" int ishmem_##NAME##_atomic_fetch_xor(int my_pe, T *fetched_host, T *target, T value, int pe)       \
    {                                                                                                             \
        return host_amo<T, D>(my_pe, AMO_FETCH_XOR, fetched_host, target, value, 0, pe, true);                    \
    }
ISHMEMI_DEF_AMO(int32, int32_t, int)
ISHMEMI_DEF_AMO(int64, int64_t, long long)
ISHMEMI_DEF_AMO(uint32, uint32_t, unsigned)
ISHMEMI_DEF_AMO(uint64, uint64_t, unsigned long long)

/* ---- device-initiated batches ---------------------------------------------------------- */
/* Op i is issued by PE (i mod npes): the thread that handles it uses that PE's context for the
 * address translation.  Consecutive threads take consecutive ops (coalesced reads of the op
 * stream).  Word w lives on PE (w mod npes), slot (w div npes). */

#define AMO_BLOCK_SLOTS 2048 /* shared-memory accumulators of the block-level aggregation */
#define AMO_BLOCK_OPT 8      /* ops per thread in that mode */

__device__ __forceinline__ long long *table_of(const ishmem_ctx_t *ctxs, const ishmem_ctx_t *ctx, long long *table0)
{
    return (long long *)((char *)table0 + (ctx->heap_base - ctxs[0].heap_base));
}

/* Lanes of the warp (those in `act`) that hit the same word w combine: on return `total` is the
 * sum of the group's increments, `before` the sum over the group's lower lanes (what this lane
 * would find added already if the group's ops ran back to back in lane order), and the result
 * is the group's lowest lane, which issues the one atomic.  Called by every lane in `act`. */
__device__ __forceinline__ unsigned warp_combine(unsigned act, int w, long long v, long long *total, long long *before)
{
    const unsigned lane = threadIdx.x & 31u;
    const unsigned peers = __match_any_sync(act, w);
    long long bef = 0, tot = 0;
    unsigned rest = peers;
    /* round r: every lane reads the increment of its r-th peer; the number of rounds is the
     * largest group in the warp, so the shuffles stay converged */
    const unsigned rounds = __reduce_max_sync(act, (unsigned)__popc(peers));
#pragma unroll 1
    for (unsigned r = 0; r < rounds; ++r) {
        const unsigned src = rest ? (unsigned)(__ffs(rest) - 1) : lane;
        const long long x = __shfl_sync(act, v, src);
        if (rest) {
            tot += x;
            if (src < lane) bef += x;
            rest &= rest - 1;
        }
    }
    *total = tot;
    *before = bef;
    return (unsigned)__ffs(peers) - 1;
}

/* MODE 0: one atomic per op.  MODE 1: lanes of a warp that hit the same word combine into one
 * atomic.  MODE 2: the ops of a block (AMO_BLOCK_OPT per thread) that hit the same word combine,
 * first within each warp, then in a direct-mapped table of shared-memory accumulators; one
 * global atomic per used slot.
 * In every mode each op gets the value it would have fetched in ONE valid serialisation. */
template <int MODE>
__global__ void __launch_bounds__(1024) k_fetch_add_batch(const ishmem_ctx_t *ctxs, long long *table0,
                                                          const int *word_idx, const long long *inc,
                                                          long long *fetched, size_t nops)
{
    const int npes = ctxs[0].npes;
    if (MODE == 2) {
        __shared__ int tag[AMO_BLOCK_SLOTS];
        __shared__ unsigned long long acc[AMO_BLOCK_SLOTS];
        for (unsigned k = threadIdx.x; k < AMO_BLOCK_SLOTS; k += blockDim.x) {
            tag[k] = -1;
            acc[k] = 0ull;
        }
        __syncthreads();
        const size_t base = (size_t)blockIdx.x * blockDim.x * AMO_BLOCK_OPT;
        long long mine[AMO_BLOCK_OPT]; /* value fetched from shared memory, or from the table if direct */
        int slot[AMO_BLOCK_OPT];       /* slot used, -1: went straight to the table, -2: no op */
#pragma unroll
        for (int j = 0; j < AMO_BLOCK_OPT; ++j) {
            const size_t i = base + (size_t)j * blockDim.x + threadIdx.x;
            const bool active = i < nops;
            const unsigned act = __ballot_sync(0xffffffffu, active);
            slot[j] = -2;
            mine[j] = 0;
            if (active) {
                const int w = word_idx[i];
                const long long v = inc[i];
                long long total, before;
                const unsigned leader = warp_combine(act, w, v, &total, &before);
                long long got = 0;
                int sl = -1;
                if ((threadIdx.x & 31u) == leader) {
                    sl = w & (AMO_BLOCK_SLOTS - 1);
                    const int seen = atomicCAS(&tag[sl], -1, w);
                    if (seen == -1 || seen == w) {
                        got = (long long)atomicAdd(&acc[sl], (unsigned long long)total);
                    } else { /* slot taken by another word: the group goes to the table itself */
                        const ishmem_ctx_t *ctx = ctxs + (int)(i % (size_t)npes);
                        got = ishmem_atomic_fetch_add<long long>(ctx, table_of(ctxs, ctx, table0) + w / npes, total,
                                                                 w % npes);
                        sl = -1;
                    }
                }
                mine[j] = __shfl_sync(act, got, leader) + before;
                slot[j] = __shfl_sync(act, sl, leader);
            }
        }
        __syncthreads();
        /* one atomic per used slot carries the block's total; the slot then holds the value the
         * table had before it */
        const ishmem_ctx_t *bctx = ctxs + (int)(blockIdx.x % (unsigned)npes);
        for (unsigned k = threadIdx.x; k < AMO_BLOCK_SLOTS; k += blockDim.x) {
            const int w = tag[k];
            if (w >= 0)
                acc[k] = (unsigned long long)ishmem_atomic_fetch_add<long long>(
                    bctx, table_of(ctxs, bctx, table0) + w / npes, (long long)acc[k], w % npes);
        }
        __syncthreads();
        if (fetched) {
#pragma unroll
            for (int j = 0; j < AMO_BLOCK_OPT; ++j) {
                const size_t i = base + (size_t)j * blockDim.x + threadIdx.x;
                if (slot[j] >= 0) fetched[i] = (long long)acc[slot[j]] + mine[j];
                else if (slot[j] == -1) fetched[i] = mine[j];
            }
        }
        return;
    }
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool active = i < nops;
    const ishmem_ctx_t *ctx = ctxs + (int)(i % (size_t)npes);
    long long *table = table_of(ctxs, ctx, table0);
    int w = 0;
    long long v = 0;
    if (active) {
        w = word_idx[i];
        v = inc[i];
    }
    if (MODE == 0) {
        if (active) {
            long long old = ishmem_atomic_fetch_add<long long>(ctx, table + w / npes, v, w % npes);
            if (fetched) fetched[i] = old;
        }
        return;
    }
    /* Lanes of the warp that hit the same word combine: the lowest such lane issues one
     * atomic with the sum and every lane rebuilds the value it would have fetched had the
     * group's ops been applied back to back in lane order. */
    const unsigned lane = threadIdx.x & 31u;
    const unsigned act = __ballot_sync(0xffffffffu, active);
    if (!active) return;
    long long before = 0, total = 0;
    const unsigned leader = warp_combine(act, w, v, &total, &before);
    long long base = 0;
    if (lane == leader) base = ishmem_atomic_fetch_add<long long>(ctx, table + w / npes, total, w % npes);
    base = __shfl_sync(act, base, leader);
    if (fetched) fetched[i] = base + before;
}

/* AGGREGATE: the lanes of a warp that hit the same word act as one group whose compare-and-swaps
 * are applied back to back in lane order: the group's lowest lane reads the word, runs the chain
 * on that value (each op sees the state its predecessors left and swaps if it equals its
 * condition) and installs the end state with ONE compare-and-swap against the value it read,
 * retrying when somebody else got in between.  The successful swap (or, when the chain changes
 * nothing, the read) is the point at which the whole group takes effect. */
template <bool AGGREGATE>
__global__ void __launch_bounds__(1024) k_compare_swap_batch(const ishmem_ctx_t *ctxs, long long *table0,
                                                             const int *word_idx, const long long *cond,
                                                             const long long *value, long long *fetched,
                                                             size_t nops)
{
    const int npes = ctxs[0].npes;
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool active = i < nops;
    const ishmem_ctx_t *ctx = ctxs + (int)(i % (size_t)npes);
    long long *table = table_of(ctxs, ctx, table0);
    if (!AGGREGATE) {
        if (!active) return;
        const int w = word_idx[i];
        long long old = ishmem_atomic_compare_swap<long long>(ctx, table + w / npes, cond[i], value[i], w % npes);
        if (fetched) fetched[i] = old;
        return;
    }
    __shared__ long long sh_cond[1024], sh_val[1024], sh_old[1024];
    const unsigned lane = threadIdx.x & 31u, wbase = threadIdx.x & ~31u;
    const unsigned act = __ballot_sync(0xffffffffu, active);
    if (!active) return;
    const int w = word_idx[i];
    sh_cond[threadIdx.x] = cond[i];
    sh_val[threadIdx.x] = value[i];
    const unsigned peers = __match_any_sync(act, w);
    __syncwarp(act);
    if (lane == (unsigned)__ffs(peers) - 1) {
        long long *target = ishmem_ptr(ctx, table + w / npes, w % npes);
        if (target) {
            for (int tries = 0;; ++tries) {
                const long long cur = ishmem_atomic_fetch<long long>(ctx, table + w / npes, w % npes);
                long long state = cur;
                for (unsigned rest = peers; rest; rest &= rest - 1) {
                    const unsigned k = wbase + (unsigned)__ffs(rest) - 1;
                    sh_old[k] = state;
                    if (state == sh_cond[k]) state = sh_val[k];
                }
                if (state == cur) break; /* the chain leaves the word as it is */
                if ((long long)atomicCAS((unsigned long long *)target, (unsigned long long)cur,
                                         (unsigned long long)state) == cur)
                    break;
                if (tries == 4096) { /* give way: apply the ops one by one */
                    for (unsigned rest = peers; rest; rest &= rest - 1) {
                        const unsigned k = wbase + (unsigned)__ffs(rest) - 1;
                        sh_old[k] = (long long)atomicCAS((unsigned long long *)target, (unsigned long long)sh_cond[k],
                                                         (unsigned long long)sh_val[k]);
                    }
                    break;
                }
            }
        }
    }
    __syncwarp(act);
    if (fetched) fetched[i] = sh_old[threadIdx.x];
}

static int batch_geometry(size_t nops, int threads, int ops_per_thread, unsigned *blocks)
{
    if (threads < 32 || threads > 1024 || threads % 32) return ISHMEM_ERR_ARG;
    const size_t per_block = (size_t)threads * ops_per_thread;
    size_t b = (nops + per_block - 1) / per_block;
    if (b == 0) b = 1;
    if (b > 0x7fffffffull) return ISHMEM_ERR_ARG;
    *blocks = (unsigned)b;
    return ISHMEM_OK;
}

extern "C" int ishmemx_int64_atomic_fetch_add_batch(int64_t *table, const int32_t *word_idx, const int64_t *inc,
                                                    int64_t *fetched, size_t nops, int threads, int aggregate)
{
    ISHMEMI_REQUIRE_INIT();
    auto &g = g_ishmem;
    if (!word_idx || !inc) return ISHMEM_ERR_ARG;
    if ((uintptr_t)table % 8) return ISHMEM_ERR_ALIGN;
    if (ishmemi_sym_offset(table, 8) < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    if (aggregate < 0 || aggregate > 2) return ISHMEM_ERR_ARG;
    unsigned blocks;
    int rc = batch_geometry(nops, threads, aggregate == 2 ? AMO_BLOCK_OPT : 1, &blocks);
    if (rc) return rc;
    cudaStream_t s;
    if ((rc = ishmemi_team_stream_begin(ISHMEM_TEAM_WORLD, &s))) return rc;
    if (nops) {
        if (aggregate == 2)
            k_fetch_add_batch<2><<<blocks, threads, 0, s>>>(g.d_ctx, (long long *)table, word_idx,
                                                            (const long long *)inc, (long long *)fetched, nops);
        else if (aggregate == 1)
            k_fetch_add_batch<1><<<blocks, threads, 0, s>>>(g.d_ctx, (long long *)table, word_idx,
                                                            (const long long *)inc, (long long *)fetched, nops);
        else
            k_fetch_add_batch<0><<<blocks, threads, 0, s>>>(g.d_ctx, (long long *)table, word_idx,
                                                            (const long long *)inc, (long long *)fetched, nops);
        ishmemi_count_launch();
        rc = ishmemi_check_launch("k_fetch_add_batch");
    }
    ishmemi_team_stream_end();
    return rc;
}

extern "C" int ishmemx_int64_atomic_compare_swap_batch(int64_t *table, const int32_t *word_idx,
                                                       const int64_t *cond, const int64_t *value,
                                                       int64_t *fetched, size_t nops, int threads, int aggregate)
{
    ISHMEMI_REQUIRE_INIT();
    auto &g = g_ishmem;
    if (!word_idx || !cond || !value || aggregate < 0 || aggregate > 1) return ISHMEM_ERR_ARG;
    if ((uintptr_t)table % 8) return ISHMEM_ERR_ALIGN;
    if (ishmemi_sym_offset(table, 8) < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    unsigned blocks;
    int rc = batch_geometry(nops, threads, 1, &blocks);
    if (rc) return rc;
    cudaStream_t s;
    if ((rc = ishmemi_team_stream_begin(ISHMEM_TEAM_WORLD, &s))) return rc;
    if (nops) {
        if (aggregate)
            k_compare_swap_batch<true><<<blocks, threads, 0, s>>>(g.d_ctx, (long long *)table, word_idx,
                                                                  (const long long *)cond, (const long long *)value,
                                                                  (long long *)fetched, nops);
        else
            k_compare_swap_batch<false><<<blocks, threads, 0, s>>>(g.d_ctx, (long long *)table, word_idx,
                                                                   (const long long *)cond, (const long long *)value,
                                                                   (long long *)fetched, nops);
        ishmemi_count_launch();
        rc = ishmemi_check_launch("k_compare_swap_batch");
    }
    ishmemi_team_stream_end();
    return rc;
}
