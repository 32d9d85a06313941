/* Host runtime of libishmem.so: PE contexts, symmetric heap and allocator, streams, teams,
 * status.  Host-only work (Section 3.6 of the paper: initialisation and all memory
 * management are host calls). */
#include <cstdlib>
#include <cstring>

#include "internal.h"

ishmemi_state g_ishmem;

int ishmemi_cuda(cudaError_t e, const char *what)
{
    if (e == cudaSuccess) return ISHMEM_OK;
    g_ishmem.last_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
    (void)cudaGetLastError(); /* a refused launch must not show up again in the next call's check */
    if (e == cudaErrorCooperativeLaunchTooLarge) return ISHMEM_ERR_NOT_CORESIDENT;
    if (e == cudaErrorMemoryAllocation) return ISHMEM_ERR_OOM;
    return ISHMEM_ERR_CUDA;
}

int ishmemi_check_launch(const char *what) { return ishmemi_cuda(cudaGetLastError(), what); }
void ishmemi_count_launch(unsigned n) { g_ishmem.launches += n; }

int ishmemi_check_pe(int pe)
{
    return (pe >= 0 && pe < g_ishmem.npes) ? ISHMEM_OK : ISHMEM_ERR_INVALID_PE;
}

long long ishmemi_sym_offset(const void *p, size_t n)
{
    const char *c = (const char *)p;
    if (c < g_ishmem.base) return -1;
    size_t off = (size_t)(c - g_ishmem.base);
    if (off > g_ishmem.heap_bytes || n > g_ishmem.heap_bytes - off) return -1;
    return (long long)off;
}

char *ishmemi_localise(const void *p, size_t n, int my_pe)
{
    long long off = ishmemi_sym_offset(p, n);
    if (off < 0) return (char *)p;
    return g_ishmem.base + (size_t)my_pe * g_ishmem.heap_bytes + (size_t)off;
}

void ishmemi_push_ctx()
{
    auto &g = g_ishmem;
    for (int p = 0; p < g.npes; ++p) {
        memcpy(g.h_ctx[p].teams, g.teams, sizeof(g.teams));
        g.h_ctx[p].wait_limit_ns = g.wait_limit_ns;
        g.h_ctx[p].bcast_root_dest = g.bcast_root_dest;
    }
    cudaMemcpy(g.d_ctx, g.h_ctx, sizeof(ishmem_ctx_t) * g.npes, cudaMemcpyHostToDevice);
}

/* ---- stream ordering ---------------------------------------------------------------- */

cudaStream_t ishmemi_pe_stream_for_op(int pe)
{
    auto &g = g_ishmem;
    if (g.pe_seen_team[pe] != g.team_seq) {
        /* the event is recorded only now, when somebody needs it: it then covers everything the
         * team stream holds (at least the launch this PE has not seen), and back-to-back team
         * launches pay for no event at all */
        if (g.team_event_seq != g.team_seq) {
            cudaEventRecord(g.ev_team, g.team_stream);
            g.team_event_seq = g.team_seq;
        }
        cudaStreamWaitEvent(g.pe_stream[pe], g.ev_team, 0);
        g.pe_seen_team[pe] = g.team_seq;
    }
    g.pe_dirty[pe] = true;
    return g.pe_stream[pe];
}

static void join_engine(int pe)
{
    auto &g = g_ishmem;
    if (g.nbi_pending[pe]) {
        cudaEventRecord(g.ev_engine[pe], g.engine_stream[pe]);
        cudaStreamWaitEvent(g.pe_stream[pe], g.ev_engine[pe], 0);
        g.nbi_pending[pe] = false;
        g.pe_dirty[pe] = true;
    }
}

int ishmemi_team_stream_begin(ishmem_team_t team, cudaStream_t *out)
{
    auto &g = g_ishmem;
    if (team < 0 || team >= ISHMEM_MAX_TEAMS || !g.teams[team].valid) return ISHMEM_ERR_ARG;
    const ishmemi_team &t = g.teams[team];
    for (int i = 0; i < t.size; ++i) {
        int p = t.start + i * t.stride;
        join_engine(p);
        if (g.pe_dirty[p]) {
            cudaEventRecord(g.ev_pe[p], g.pe_stream[p]);
            cudaStreamWaitEvent(g.team_stream, g.ev_pe[p], 0);
            g.pe_dirty[p] = false;
        }
    }
    *out = g.team_stream;
    return ISHMEM_OK;
}

void ishmemi_team_stream_end()
{
    ++g_ishmem.team_seq; /* PE streams order themselves after it lazily (ishmemi_pe_stream_for_op) */
}

int ishmemi_engine_copy(int my_pe, void *dst, const void *src, size_t n, bool blocking)
{
    auto &g = g_ishmem;
    cudaStream_t ps = ishmemi_pe_stream_for_op(my_pe);
    /* the engine starts after everything already enqueued by this PE */
    ISHMEMI_CUDA(cudaEventRecord(g.ev_pe[my_pe], ps));
    ISHMEMI_CUDA(cudaStreamWaitEvent(g.engine_stream[my_pe], g.ev_pe[my_pe], 0));
    ISHMEMI_CUDA(cudaMemcpyAsync(dst, src, n, cudaMemcpyDeviceToDevice, g.engine_stream[my_pe]));
    if (blocking) {
        ISHMEMI_CUDA(cudaEventRecord(g.ev_engine[my_pe], g.engine_stream[my_pe]));
        ISHMEMI_CUDA(cudaStreamWaitEvent(ps, g.ev_engine[my_pe], 0));
    } else {
        g.nbi_pending[my_pe] = true;
    }
    return ISHMEM_OK;
}

/* ---- lifecycle -------------------------------------------------------------------------- */

/* a size from the environment: a number of bytes (0x.. accepted), or "never" / "always" */
static bool env_size(const char *name, size_t *out)
{
    const char *v = getenv(name);
    if (!v || !*v) return false;
    if (!strcmp(v, "never")) *out = (size_t)-1;
    else if (!strcmp(v, "always")) *out = 0;
    else *out = (size_t)strtoull(v, nullptr, 0);
    return true;
}

static int init_common(int npes, size_t heap_bytes, void *external)
{
    auto &g = g_ishmem;
    if (g.initialised) return ISHMEM_ERR_ARG;
    /* ishmem_init(npes, 0): the heap size comes from ISHMEM_SYMMETRIC_SIZE (bytes per PE) */
    if (heap_bytes == 0 && !external) env_size("ISHMEM_SYMMETRIC_SIZE", &heap_bytes);
    if (npes < 1 || npes > ISHMEM_MAX_PES || heap_bytes == 0 || heap_bytes == (size_t)-1) return ISHMEM_ERR_ARG;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) {
        g.last_cuda_error = "no CUDA device: this library has no CPU path";
        return ISHMEM_ERR_CUDA;
    }
    ISHMEMI_CUDA(cudaGetDevice(&g.device));
    cudaDeviceProp prop;
    ISHMEMI_CUDA(cudaGetDeviceProperties(&prop, g.device));
    g.sm_count = prop.multiProcessorCount;
    g.max_dyn_smem = prop.sharedMemPerBlockOptin;
    heap_bytes = (heap_bytes + ISHMEMI_ALIGN - 1) / ISHMEMI_ALIGN * ISHMEMI_ALIGN;
    if (external) {
        if (((uintptr_t)external) % ISHMEMI_ALIGN) return ISHMEM_ERR_ALIGN;
        g.base = (char *)external;
        g.owns_heap = false;
    } else {
        void *p = nullptr;
        ISHMEMI_CUDA(cudaMalloc(&p, heap_bytes * (size_t)npes));
        ISHMEMI_CUDA(cudaMemset(p, 0, heap_bytes * (size_t)npes));
        g.base = (char *)p;
        g.owns_heap = true;
    }
    g.npes = npes;
    g.heap_bytes = heap_bytes;
    size_t internal = (size_t)npes * ISHMEMI_INTERNAL_BYTES + 256;
    ISHMEMI_CUDA(cudaMalloc((void **)&g.d_internal, internal));
    ISHMEMI_CUDA(cudaMemset(g.d_internal, 0, internal));
    g.d_status = (int *)(g.d_internal + (size_t)npes * ISHMEMI_INTERNAL_BYTES);
    ISHMEMI_CUDA(cudaMalloc((void **)&g.d_ctx, sizeof(ishmem_ctx_t) * npes));
    ISHMEMI_CUDA(cudaHostAlloc(&g.h_pinned, 4096, cudaHostAllocDefault));

    memset(g.teams, 0, sizeof(g.teams));
    g.teams[ISHMEM_TEAM_WORLD] = {0, 1, npes, 1};
    g.teams[ISHMEM_TEAM_SHARED] = {0, 1, npes, 1};
    for (int p = 0; p < npes; ++p) {
        ishmem_ctx_t &c = g.h_ctx[p];
        memset(&c, 0, sizeof(c));
        c.my_pe = p;
        c.npes = npes;
        c.heap_bytes = heap_bytes;
        c.heap_base = g.base + (size_t)p * heap_bytes;
        for (int q = 0; q < npes; ++q) {
            /* every PE is reachable by load/store (non-zero flag); the offset array holds
             * heap_base[q] - heap_base[p] under the same index */
            c.reach[q] = 1;
            c.heap_delta[q] = ((long long)q - (long long)p) * (long long)heap_bytes;
        }
        char *mine = g.d_internal + (size_t)p * ISHMEMI_INTERNAL_BYTES;
        c.sync_arrive = (unsigned long long *)mine;
        c.sync_epoch = (unsigned long long *)(mine + 8 * ISHMEM_MAX_TEAMS);
        c.collect_sizes = (unsigned long long *)(mine + 16 * ISHMEM_MAX_TEAMS);
        c.internal_stride = ISHMEMI_INTERNAL_BYTES;
        c.status = g.d_status;
    }
    for (int p = 0; p < npes; ++p) {
        ISHMEMI_CUDA(cudaStreamCreateWithFlags(&g.pe_stream[p], cudaStreamNonBlocking));
        g.owns_pe_stream[p] = true;
        ISHMEMI_CUDA(cudaStreamCreateWithFlags(&g.engine_stream[p], cudaStreamNonBlocking));
        ISHMEMI_CUDA(cudaEventCreateWithFlags(&g.ev_pe[p], cudaEventDisableTiming));
        ISHMEMI_CUDA(cudaEventCreateWithFlags(&g.ev_engine[p], cudaEventDisableTiming));
        g.pe_dirty[p] = false;
        g.nbi_pending[p] = false;
        g.pe_seen_team[p] = 0;
    }
    ISHMEMI_CUDA(cudaStreamCreateWithFlags(&g.team_stream, cudaStreamNonBlocking));
    g.owns_team_stream = true;
    ISHMEMI_CUDA(cudaEventCreateWithFlags(&g.ev_team, cudaEventDisableTiming));
    g.team_seq = 0;
    g.team_event_seq = 0;
    g.free_blocks.clear();
    g.used_blocks.clear();
    g.free_blocks[0] = heap_bytes;
    /* default cutovers, from the committed size sweep on B200 (ishmemx_tune_cutover re-measures):
     * a host-initiated put/get of one PE is faster on the copy engine from 4 to 32 MiB (5.9 against
     * 6.2 us at 4 MiB, 9.3 against 12.3 us at 32 MiB, back-to-back calls), slower at 64 MiB (24.7
     * against 20.6 us) and level with the tiled kernel above that: the engine's range is a band,
     * [4 MiB, 64 MiB); the push collectives and the device-initiated work-group calls never gain,
     * so they stay on loads and stores */
    g.cutover[0] = (size_t)4 << 20;
    g.cutover_put_upto = (size_t)64 << 20;
    g.cutover[1] = g.cutover[2] = g.wg_cutover = (size_t)-1;
    env_size("ISHMEM_CUTOVER_PUT", &g.cutover[0]);
    env_size("ISHMEM_CUTOVER_PUT_UPTO", &g.cutover_put_upto);
    env_size("ISHMEM_CUTOVER_BCAST", &g.cutover[1]);
    env_size("ISHMEM_CUTOVER_FCOLLECT", &g.cutover[2]);
    env_size("ISHMEM_CUTOVER_WORK_GROUP", &g.wg_cutover);
    {
        size_t ns = 0;
        if (env_size("ISHMEM_WAIT_TIMEOUT_NS", &ns) && ns && ns != (size_t)-1) g.wait_limit_ns = ns;
    }
    /* launch-shape switches: defaults, then the environment's initial values (read here only) */
    g.opt[ISHMEMX_OPT_JACOBI_SPLIT] = 0;
    g.opt[ISHMEMX_OPT_JACOBI_FUSE] = 1;
    g.opt[ISHMEMX_OPT_JACOBI_WIDE] = -1;
    g.opt[ISHMEMX_OPT_REDUCE_BULK] = 0;
    g.opt[ISHMEMX_OPT_BULK_SMEM] = 192 * 1024 + 128;
    g.opt[ISHMEMX_OPT_PUSH_SHAPE] = 0;
    if (const char *v = getenv("ISHMEM_PUSH_SHAPE")) {
        const int f = atoi(v);
        if (f >= 0 && f <= 2) g.opt[ISHMEMX_OPT_PUSH_SHAPE] = f;
    }
    if (const char *v = getenv("ISHMEM_JACOBI_SPLIT")) {
        if (!strcmp(v, "rows")) g.opt[ISHMEMX_OPT_JACOBI_SPLIT] = 1;
        else if (!strcmp(v, "columns")) g.opt[ISHMEMX_OPT_JACOBI_SPLIT] = 2;
    }
    if (const char *v = getenv("ISHMEM_JACOBI_FUSE")) {
        const int f = atoi(v);
        if (f >= 0 && f <= 6) g.opt[ISHMEMX_OPT_JACOBI_FUSE] = f;
    }
    if (const char *v = getenv("ISHMEM_JACOBI_WIDE")) g.opt[ISHMEMX_OPT_JACOBI_WIDE] = atoi(v) != 0;
    if (const char *v = getenv("ISHMEM_REDUCE_BULK")) g.opt[ISHMEMX_OPT_REDUCE_BULK] = atoi(v) != 0;
    {
        size_t b = 0;
        if (env_size("ISHMEM_BULK_SMEM", &b) && b >= 128 + 2048 && b != (size_t)-1) g.opt[ISHMEMX_OPT_BULK_SMEM] = (long long)b;
    }
    g.hybrid_head = 0;
    g.launches = 0;
    g.initialised = true;
    ishmemi_push_ctx();
    ISHMEMI_CUDA(cudaDeviceSynchronize());
    return ISHMEM_OK;
}

extern "C" int ishmem_init(int npes, size_t heap_bytes) { return init_common(npes, heap_bytes, nullptr); }

extern "C" int ishmemx_init_external(int npes, size_t heap_bytes, void *base)
{
    if (!base) return ISHMEM_ERR_ARG;
    if (heap_bytes % ISHMEMI_ALIGN) return ISHMEM_ERR_ALIGN;
    return init_common(npes, heap_bytes, base);
}

extern "C" int ishmem_finalize(void)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    cudaDeviceSynchronize();
    ishmemi_proxy_finalize();
    for (int p = 0; p < g.npes; ++p) {
        if (g.owns_pe_stream[p]) cudaStreamDestroy(g.pe_stream[p]);
        cudaStreamDestroy(g.engine_stream[p]);
        cudaEventDestroy(g.ev_pe[p]);
        cudaEventDestroy(g.ev_engine[p]);
    }
    if (g.owns_team_stream) cudaStreamDestroy(g.team_stream);
    cudaEventDestroy(g.ev_team);
    if (g.owns_heap) cudaFree(g.base);
    cudaFree(g.d_internal);
    cudaFree(g.d_ctx);
    cudaFreeHost(g.h_pinned);
    g.base = nullptr;
    g.d_internal = nullptr;
    g.d_ctx = nullptr;
    g.h_pinned = nullptr;
    g.free_blocks.clear();
    g.used_blocks.clear();
    g.npes = 0;
    g.initialised = false;
    return ISHMEM_OK;
}

extern "C" int ishmem_n_pes(void) { return g_ishmem.initialised ? g_ishmem.npes : 0; }
extern "C" size_t ishmemx_heap_bytes(void) { return g_ishmem.initialised ? g_ishmem.heap_bytes : 0; }

extern "C" void *ishmemx_ctx(int pe)
{
    if (!g_ishmem.initialised || ishmemi_check_pe(pe)) return nullptr;
    return g_ishmem.d_ctx + pe;
}

extern "C" int ishmemx_set_stream(int pe, void *cuda_stream)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    if (pe == -1) {
        ISHMEMI_CUDA(cudaStreamSynchronize(g.team_stream));
        if (g.owns_team_stream) cudaStreamDestroy(g.team_stream);
        g.team_stream = (cudaStream_t)cuda_stream;
        g.owns_team_stream = false;
        return ISHMEM_OK;
    }
    if (ishmemi_check_pe(pe)) return ISHMEM_ERR_INVALID_PE;
    ISHMEMI_CUDA(cudaStreamSynchronize(g.pe_stream[pe]));
    if (g.owns_pe_stream[pe]) cudaStreamDestroy(g.pe_stream[pe]);
    g.pe_stream[pe] = (cudaStream_t)cuda_stream;
    g.owns_pe_stream[pe] = false;
    return ISHMEM_OK;
}

extern "C" void *ishmemx_get_stream(int pe)
{
    auto &g = g_ishmem;
    if (!g.initialised) return nullptr;
    if (pe == -1) return (void *)g.team_stream;
    if (ishmemi_check_pe(pe)) return nullptr;
    return (void *)g.pe_stream[pe];
}

extern "C" const char *ishmem_strerror(int status)
{
    switch (status) {
    case ISHMEM_OK: return "success";
    case ISHMEM_ERR_INVALID_PE: return "invalid PE";
    case ISHMEM_ERR_NOT_SYMMETRIC: return "address range is not in the symmetric heap";
    case ISHMEM_ERR_ALIGN: return "misaligned address";
    case ISHMEM_ERR_OOM: return "out of memory";
    case ISHMEM_ERR_TIMEOUT: return "a bounded device-side wait timed out";
    case ISHMEM_ERR_NOT_CORESIDENT: return "launch does not fit co-resident on the device";
    case ISHMEM_ERR_CUDA: return "CUDA runtime error";
    case ISHMEM_ERR_ARG: return "invalid argument";
    case ISHMEM_ERR_NOT_INITIALIZED: return "library not initialised";
    default: return "unknown status";
    }
}

extern "C" const char *ishmemx_last_cuda_error(void) { return g_ishmem.last_cuda_error.c_str(); }

extern "C" int ishmemx_status(int clear)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    ISHMEMI_CUDA(cudaDeviceSynchronize());
    int st = 0;
    ISHMEMI_CUDA(cudaMemcpy(&st, g.d_status, sizeof(int), cudaMemcpyDeviceToHost));
    if (clear && st) ISHMEMI_CUDA(cudaMemset(g.d_status, 0, sizeof(int)));
    return st;
}

extern "C" int ishmemx_set_wait_limit_ns(uint64_t ns)
{
    ISHMEMI_REQUIRE_INIT();
    if (ns == 0) return ISHMEM_ERR_ARG;
    ISHMEMI_CUDA(cudaDeviceSynchronize());
    g_ishmem.wait_limit_ns = ns;
    ishmemi_push_ctx();
    return ISHMEM_OK;
}

extern "C" unsigned long long ishmemx_launch_count(void) { return g_ishmem.launches; }

/* ---- symmetric allocator: first fit over a sorted free list, coalescing on free ----------- */

static void *sym_alloc(size_t alignment, size_t size)
{
    auto &g = g_ishmem;
    if (!g.initialised || size == 0) return nullptr;
    if (alignment < ISHMEMI_ALIGN) alignment = ISHMEMI_ALIGN;
    if (alignment & (alignment - 1)) return nullptr;
    size_t need = (size + ISHMEMI_ALIGN - 1) / ISHMEMI_ALIGN * ISHMEMI_ALIGN;
    if (need < size) return nullptr;
    std::lock_guard<std::mutex> lk(g.mu);
    for (auto it = g.free_blocks.begin(); it != g.free_blocks.end(); ++it) {
        size_t off = it->first, len = it->second;
        /* alignment is relative to the device address; heap bases are 256-byte aligned */
        uintptr_t addr = (uintptr_t)g.base + off;
        size_t pad = (size_t)((alignment - addr % alignment) % alignment);
        if (pad > len || need > len - pad) continue;
        size_t start = off + pad;
        g.free_blocks.erase(it);
        if (pad) g.free_blocks[off] = pad;
        if (len - pad - need) g.free_blocks[start + need] = len - pad - need;
        g.used_blocks[start] = need;
        return g.base + start;
    }
    return nullptr;
}

extern "C" void *ishmem_malloc(size_t size) { return sym_alloc(ISHMEMI_ALIGN, size); }
extern "C" void *ishmem_align(size_t alignment, size_t size) { return sym_alloc(alignment, size); }

extern "C" void *ishmem_calloc(size_t count, size_t size)
{
    auto &g = g_ishmem;
    if (size && count > (size_t)-1 / size) return nullptr;
    void *p = sym_alloc(ISHMEMI_ALIGN, count * size);
    if (!p) return nullptr;
    size_t off = (size_t)((char *)p - g.base);
    /* The zeroing is one world-team operation: it waits for every PE's earlier work and every PE
     * stream orders its later work after it, so a put or atomic that some PE issues right after
     * the call cannot be overtaken by another PE's clearing (OpenSHMEM's calloc ends with a
     * barrier for the same reason). */
    cudaStream_t s;
    if (ishmemi_team_stream_begin(ISHMEM_TEAM_WORLD, &s)) {
        ishmem_free(p);
        return nullptr;
    }
    bool ok = true;
    for (int pe = 0; pe < g.npes && ok; ++pe)
        ok = cudaMemsetAsync(g.base + (size_t)pe * g.heap_bytes + off, 0, count * size, s) == cudaSuccess;
    ishmemi_team_stream_end();
    if (!ok) {
        (void)cudaGetLastError();
        ishmem_free(p);
        return nullptr;
    }
    return p;
}

extern "C" int ishmem_free(void *ptr)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    if (!ptr) return ISHMEM_OK;
    std::lock_guard<std::mutex> lk(g.mu);
    long long off = ishmemi_sym_offset(ptr, 0);
    if (off < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    auto it = g.used_blocks.find((size_t)off);
    if (it == g.used_blocks.end()) return ISHMEM_ERR_ARG;
    size_t start = it->first, len = it->second;
    g.used_blocks.erase(it);
    auto next = g.free_blocks.lower_bound(start);
    if (next != g.free_blocks.end() && next->first == start + len) {
        len += next->second;
        next = g.free_blocks.erase(next);
    }
    if (next != g.free_blocks.begin()) {
        auto prev = std::prev(next);
        if (prev->first + prev->second == start) {
            prev->second += len;
            return ISHMEM_OK;
        }
    }
    g.free_blocks[start] = len;
    return ISHMEM_OK;
}

extern "C" void *ishmem_ptr(const void *sym, int pe)
{
    auto &g = g_ishmem;
    if (!g.initialised || ishmemi_check_pe(pe)) return nullptr;
    long long off = ishmemi_sym_offset(sym, 0);
    if (off < 0) return nullptr;
    return g.base + (size_t)pe * g.heap_bytes + (size_t)off;
}

extern "C" int ishmemx_heap_write(int pe, void *sym_dest, const void *host, size_t nbytes)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    if (ishmemi_check_pe(pe)) return ISHMEM_ERR_INVALID_PE;
    long long off = ishmemi_sym_offset(sym_dest, nbytes);
    if (off < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    cudaStream_t s = ishmemi_pe_stream_for_op(pe);
    ISHMEMI_CUDA(cudaMemcpyAsync(g.base + (size_t)pe * g.heap_bytes + (size_t)off, host, nbytes,
                                 cudaMemcpyHostToDevice, s));
    return ISHMEM_OK;
}

extern "C" int ishmemx_heap_read(int pe, void *host, const void *sym_src, size_t nbytes)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    if (ishmemi_check_pe(pe)) return ISHMEM_ERR_INVALID_PE;
    long long off = ishmemi_sym_offset(sym_src, nbytes);
    if (off < 0) return ISHMEM_ERR_NOT_SYMMETRIC;
    cudaStream_t s = ishmemi_pe_stream_for_op(pe);
    ISHMEMI_CUDA(cudaMemcpyAsync(host, g.base + (size_t)pe * g.heap_bytes + (size_t)off, nbytes,
                                 cudaMemcpyDeviceToHost, s));
    return ISHMEM_OK;
}

/* ---- teams ---------------------------------------------------------------------------------- */

extern "C" ishmem_team_t ishmem_team_split_strided(ishmem_team_t parent, int start, int stride, int size)
{
    auto &g = g_ishmem;
    if (!g.initialised || parent < 0 || parent >= ISHMEM_MAX_TEAMS || !g.teams[parent].valid)
        return ISHMEM_TEAM_INVALID;
    const ishmemi_team pt = g.teams[parent];
    if (size < 1 || stride < 1 || start < 0 || start + (size - 1) * stride >= pt.size)
        return ISHMEM_TEAM_INVALID;
    for (int t = 2; t < ISHMEM_MAX_TEAMS; ++t)
        if (!g.teams[t].valid) {
            cudaDeviceSynchronize();
            g.teams[t] = {pt.start + start * pt.stride, stride * pt.stride, size, 1};
            /* a recycled slot starts from fresh counters on every PE */
            for (int p = 0; p < g.npes; ++p) {
                cudaMemset(g.h_ctx[p].sync_arrive + t, 0, 8);
                cudaMemset(g.h_ctx[p].sync_epoch + t, 0, 8);
            }
            ishmemi_push_ctx();
            return t;
        }
    return ISHMEM_TEAM_INVALID;
}

extern "C" int ishmem_team_split_2d(ishmem_team_t parent, int xrange, int parent_index, ishmem_team_t *xaxis_team,
                                    ishmem_team_t *yaxis_team)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    if (parent < 0 || parent >= ISHMEM_MAX_TEAMS || !g.teams[parent].valid || !xaxis_team || !yaxis_team)
        return ISHMEM_ERR_ARG;
    const int size = g.teams[parent].size;
    if (xrange < 1 || parent_index < 0 || parent_index >= size) return ISHMEM_ERR_ARG;
    if (xrange > size) xrange = size;
    const int x = parent_index % xrange, y = parent_index / xrange;
    const int row_size = (size - y * xrange) < xrange ? size - y * xrange : xrange;
    const int col_size = (size - x + xrange - 1) / xrange;
    ishmem_team_t tx = ishmem_team_split_strided(parent, y * xrange, 1, row_size);
    if (tx == ISHMEM_TEAM_INVALID) return ISHMEM_ERR_ARG;
    ishmem_team_t ty = ishmem_team_split_strided(parent, x, xrange, col_size);
    if (ty == ISHMEM_TEAM_INVALID) {
        ishmem_team_destroy(tx);
        return ISHMEM_ERR_ARG;
    }
    *xaxis_team = tx;
    *yaxis_team = ty;
    return ISHMEM_OK;
}

extern "C" int ishmem_team_destroy(ishmem_team_t team)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    if (team < 2 || team >= ISHMEM_MAX_TEAMS || !g.teams[team].valid) return ISHMEM_ERR_ARG;
    cudaDeviceSynchronize();
    g.teams[team].valid = 0;
    ishmemi_push_ctx();
    return ISHMEM_OK;
}

extern "C" int ishmem_team_n_pes(ishmem_team_t team)
{
    auto &g = g_ishmem;
    if (!g.initialised || team < 0 || team >= ISHMEM_MAX_TEAMS || !g.teams[team].valid) return -1;
    return g.teams[team].size;
}

static int index_in(const ishmemi_team &t, int pe)
{
    const int d = pe - t.start;
    if (d < 0 || d % t.stride) return -1;
    return d / t.stride < t.size ? d / t.stride : -1;
}
extern "C" int ishmem_team_my_pe(ishmem_team_t team, int pe)
{
    auto &g = g_ishmem;
    if (!g.initialised || team < 0 || team >= ISHMEM_MAX_TEAMS || !g.teams[team].valid || ishmemi_check_pe(pe)) return -1;
    return index_in(g.teams[team], pe);
}
extern "C" int ishmem_team_translate_pe(ishmem_team_t src_team, int src_pe, ishmem_team_t dest_team)
{
    auto &g = g_ishmem;
    if (!g.initialised || src_team < 0 || src_team >= ISHMEM_MAX_TEAMS || !g.teams[src_team].valid) return -1;
    if (dest_team < 0 || dest_team >= ISHMEM_MAX_TEAMS || !g.teams[dest_team].valid) return -1;
    const ishmemi_team &s = g.teams[src_team];
    if (src_pe < 0 || src_pe >= s.size) return -1;
    return index_in(g.teams[dest_team], s.start + src_pe * s.stride);
}
extern "C" void ishmem_info_get_version(int *major, int *minor)
{
    if (major) *major = ISHMEM_MAJOR_VERSION;
    if (minor) *minor = ISHMEM_MINOR_VERSION;
}
extern "C" void ishmem_info_get_name(char *name)
{
    if (name) strncpy(name, "ishmem for B200 (sm_100a), after Intel SHMEM", ISHMEM_MAX_NAME_LEN - 1), name[ISHMEM_MAX_NAME_LEN - 1] = 0;
}

extern "C" int ishmemx_set_cutover(int which, size_t nbytes)
{
    ISHMEMI_REQUIRE_INIT();
    if (which < 0 || which > 5) return ISHMEM_ERR_ARG;
    if (which == 5) {
        g_ishmem.cutover_put_upto = nbytes;
        return ISHMEM_OK;
    }
    if (which >= 3) {
        if (which == 3) g_ishmem.wg_cutover = nbytes;
        else g_ishmem.hybrid_head = nbytes;
        ishmemi_proxy_set_cutover(g_ishmem.wg_cutover, g_ishmem.hybrid_head);
        return ISHMEM_OK;
    }
    g_ishmem.cutover[which] = nbytes;
    return ISHMEM_OK;
}
extern "C" size_t ishmemx_get_cutover(int which)
{
    if (which == 3) return g_ishmem.wg_cutover;
    if (which == 4) return g_ishmem.hybrid_head;
    if (which == 5) return g_ishmem.cutover_put_upto;
    return (which < 0 || which > 2) ? 0 : g_ishmem.cutover[which];
}
extern "C" int ishmemx_set_option(int option, long long value)
{
    ISHMEMI_REQUIRE_INIT();
    switch (option) {
    case ISHMEMX_OPT_JACOBI_SPLIT:
    case ISHMEMX_OPT_PUSH_SHAPE:
        if (value < 0 || value > 2) return ISHMEM_ERR_ARG;
        break;
    case ISHMEMX_OPT_JACOBI_FUSE:
        if (value < 0 || value > 6) return ISHMEM_ERR_ARG;
        break;
    case ISHMEMX_OPT_REDUCE_BULK:
        if (value < 0 || value > 1) return ISHMEM_ERR_ARG;
        break;
    case ISHMEMX_OPT_JACOBI_WIDE:
        if (value < -1 || value > 1) return ISHMEM_ERR_ARG;
        break;
    case ISHMEMX_OPT_BULK_SMEM:
        if (value < 128 + 2048 || value > (1 << 20)) return ISHMEM_ERR_ARG;
        break;
    default: return ISHMEM_ERR_ARG;
    }
    g_ishmem.opt[option] = value;
    return ISHMEM_OK;
}
extern "C" long long ishmemx_get_option(int option)
{
    return (option < 0 || option >= ISHMEMX_OPT_COUNT) ? 0 : g_ishmem.opt[option];
}
extern "C" int ishmemx_set_bcast_root_dest(int enable)
{
    ISHMEMI_REQUIRE_INIT();
    cudaDeviceSynchronize();
    g_ishmem.bcast_root_dest = enable ? 1 : 0;
    ishmemi_push_ctx();
    return ISHMEM_OK;
}
extern "C" int ishmemx_set_collective_geometry(int groups_per_pe, int threads)
{
    ISHMEMI_REQUIRE_INIT();
    if (groups_per_pe < 0 || threads < 32 || threads > 1024 || threads % 32) return ISHMEM_ERR_ARG;
    g_ishmem.coll_groups = groups_per_pe;
    g_ishmem.coll_threads = threads;
    return ISHMEM_OK;
}
