/* Reverse offload (Section 3.4 of the paper, "Synchronization with Host"): GPU threads post
 * fixed-size requests into a lock-free ring in pinned host memory; one host thread serves them
 * the way it would serve operations started on the host (Section 3.7.1) -- here: it starts the
 * copy engine for device-initiated puts and gets above the cutover.
 *
 * Both directions use stores only.  GPU -> host: the message, then its sequence number with a
 * system-scope release.  Host -> GPU: replies are 64-bit words in pinned host memory that the
 * waiting GPU thread polls; a reply that must follow a copy is written by the copy-engine
 * stream itself (a stream memory operation placed after the copy), so the proxy thread never
 * waits for the GPU.  Flow control is a tail counter that the proxy publishes every few
 * messages and that GPU threads read only when the ring looks full. */
#include <atomic>
#include <chrono>
#include <cstring>
#include <thread>

#include <cuda.h>

#include "internal.h"

#define PROXY_RING_SLOTS 8192u
#define PROXY_COMP_SLOTS 65536u

typedef CUresult (*write_value64_fn)(CUstream, CUdeviceptr, cuuint64_t, unsigned int);

struct proxy_state {
    bool running = false;
    std::thread thread;
    std::atomic<bool> stop{false};
    /* pinned host memory */
    ishmemi_request *ring = nullptr;
    unsigned long long *host_words = nullptr; /* [0]: tail_pub, [8 ..): nbi_done[npes], then comp[] */
    unsigned long long *tail_pub = nullptr, *nbi_done = nullptr, *comp = nullptr;
    unsigned long long *values = nullptr;     /* source words of in-stream replies when stream memory
                                                 operations are unavailable */
    /* device memory */
    unsigned long long *d_words = nullptr;    /* head, tail_cache, comp_alloc, nbi_issued[npes], nbi_seen[npes] */
    ishmemi_proxy_t *d_proxy = nullptr;
    ishmemi_proxy_t h_proxy = {};
    write_value64_fn write64 = nullptr;
    unsigned long long nbi_count[ISHMEM_MAX_PES] = {};
    std::atomic<unsigned long long> served{0}, copies{0};
    std::atomic<int> error{0};
};
static proxy_state g_px;

/* reply `value` into the pinned word `word`, ordered after everything already in `s` */
static int reply_in_stream(cudaStream_t s, unsigned long long *word, unsigned long long value, unsigned long long slot)
{
    if (g_px.write64) {
        CUresult r = g_px.write64((CUstream)s, (CUdeviceptr)(uintptr_t)word, (cuuint64_t)value, 0);
        return r == CUDA_SUCCESS ? 0 : ISHMEM_ERR_CUDA;
    }
    unsigned long long *v = g_px.values + (slot & (PROXY_COMP_SLOTS - 1));
    *v = value;
    return cudaMemcpyAsync(word, v, 8, cudaMemcpyDefault, s) == cudaSuccess ? 0 : ISHMEM_ERR_CUDA;
}

static void proxy_main(int device)
{
    auto &g = g_ishmem;
    cudaSetDevice(device);
    unsigned long long tail = 0, published = 0;
    unsigned idle = 0;
    while (!g_px.stop.load(std::memory_order_acquire)) {
        ishmemi_request *slot = g_px.ring + (tail & (PROXY_RING_SLOTS - 1));
        const unsigned long long seq = __atomic_load_n(&slot->seq, __ATOMIC_ACQUIRE);
        if (seq != tail + 1) {
            /* nothing new: make the consumed slots available, then back off a little */
            if (published != tail) {
                __atomic_store_n(g_px.tail_pub, tail, __ATOMIC_RELEASE);
                published = tail;
            }
            if (++idle > 2000) std::this_thread::sleep_for(std::chrono::microseconds(20));
            else if (idle > 200) std::this_thread::yield();
            continue;
        }
        idle = 0;
        const ishmemi_request r = *slot;
        ++tail;
        __builtin_prefetch(g_px.ring + ((tail + 4) & (PROXY_RING_SLOTS - 1)));
        if (tail - published >= PROXY_RING_SLOTS / 8) {
            __atomic_store_n(g_px.tail_pub, tail, __ATOMIC_RELEASE);
            published = tail;
        }
        int rc = 0;
        const int pe = (int)r.pe < g.npes ? (int)r.pe : 0;
        cudaStream_t s = g.engine_stream[pe];
        if (r.op == ISHMEMI_REQ_COPY || r.op == ISHMEMI_REQ_COPY_SIGNAL) {
            if (cudaMemcpyAsync((void *)(uintptr_t)r.dest, (const void *)(uintptr_t)r.src, (size_t)r.nbytes,
                                cudaMemcpyDeviceToDevice, s) != cudaSuccess)
                rc = ISHMEM_ERR_CUDA;
            if (!rc && r.op == ISHMEMI_REQ_COPY_SIGNAL) {
                /* the signal word is device memory: an 8-byte copy from a pinned source keeps it
                 * behind the payload in stream order whether or not stream memory operations exist */
                rc = reply_in_stream(s, (unsigned long long *)(uintptr_t)r.sig_addr, r.sig_value, tail);
            }
            g_px.copies.fetch_add(1, std::memory_order_relaxed);
            /* A copy that could not be started never raises its signal (the waiter must not see a
             * signal without its payload), but the request still completes, in stream order like
             * every other reply of this PE, so that the requester's wait or quiet ends at once
             * instead of by its time limit; the failure is kept for ishmemx_proxy_stop to report. */
            const int rc_copy = rc;
            rc = r.completion ? reply_in_stream(s, g_px.comp + ((r.completion - 1) & (PROXY_COMP_SLOTS - 1)), r.completion, tail)
                              : reply_in_stream(s, g_px.nbi_done + pe, ++g_px.nbi_count[pe], tail);
            if (rc_copy) rc = rc_copy;
        } else if (r.completion) {
            /* ISHMEMI_REQ_NOP: the reply is a plain store into the polled word */
            __atomic_store_n(&g_px.comp[(r.completion - 1) & (PROXY_COMP_SLOTS - 1)], r.completion, __ATOMIC_RELEASE);
        }
        if (rc) {
            (void)cudaGetLastError();
            g_px.error.store(rc, std::memory_order_relaxed);
        }
        g_px.served.store(tail, std::memory_order_relaxed); /* only this thread writes it */
    }
    __atomic_store_n(g_px.tail_pub, tail, __ATOMIC_RELEASE);
}

static void proxy_release()
{
    if (g_px.ring) cudaFreeHost(g_px.ring);
    if (g_px.host_words) cudaFreeHost(g_px.host_words);
    if (g_px.values) cudaFreeHost(g_px.values);
    if (g_px.d_words) cudaFree(g_px.d_words);
    if (g_px.d_proxy) cudaFree(g_px.d_proxy);
    g_px.ring = nullptr;
    g_px.host_words = g_px.values = nullptr;
    g_px.d_words = nullptr;
    g_px.d_proxy = nullptr;
}

extern "C" int ishmemx_proxy_start(void)
{
    ISHMEMI_REQUIRE_INIT();
    auto &g = g_ishmem;
    if (g_px.running) return ISHMEM_OK;
    ISHMEMI_CUDA(cudaDeviceSynchronize());
    const size_t host_words = 8 + ISHMEM_MAX_PES + PROXY_COMP_SLOTS;
    const size_t dev_words = 8 + 2 * ISHMEM_MAX_PES + 8; /* the last 8: results of the ring benchmark */
    int rc = ishmemi_cuda(cudaHostAlloc((void **)&g_px.ring, sizeof(ishmemi_request) * PROXY_RING_SLOTS,
                                        cudaHostAllocMapped | cudaHostAllocPortable),
                          "cudaHostAlloc(ring)");
    if (!rc) rc = ishmemi_cuda(cudaHostAlloc((void **)&g_px.host_words, 8 * host_words,
                                             cudaHostAllocMapped | cudaHostAllocPortable), "cudaHostAlloc(words)");
    if (!rc) rc = ishmemi_cuda(cudaHostAlloc((void **)&g_px.values, 8 * PROXY_COMP_SLOTS, cudaHostAllocPortable),
                               "cudaHostAlloc(values)");
    if (!rc) rc = ishmemi_cuda(cudaMalloc((void **)&g_px.d_words, 8 * dev_words), "cudaMalloc(proxy words)");
    if (!rc) rc = ishmemi_cuda(cudaMalloc((void **)&g_px.d_proxy, sizeof(ishmemi_proxy_t)), "cudaMalloc(proxy)");
    if (!rc) rc = ishmemi_cuda(cudaMemset(g_px.d_words, 0, 8 * dev_words), "cudaMemset(proxy words)");
    if (rc) {
        proxy_release();
        return rc;
    }
    memset(g_px.ring, 0, sizeof(ishmemi_request) * PROXY_RING_SLOTS);
    memset(g_px.host_words, 0, 8 * host_words);
    g_px.tail_pub = g_px.host_words;
    g_px.nbi_done = g_px.host_words + 8;
    g_px.comp = g_px.host_words + 8 + ISHMEM_MAX_PES;
    for (int p = 0; p < ISHMEM_MAX_PES; ++p) g_px.nbi_count[p] = 0;
    /* stream memory operations let the engine stream write a reply itself */
    g_px.write64 = nullptr;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuStreamWriteValue64", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess && fn && !getenv("ISHMEM_PROXY_NO_STREAM_MEMOPS"))
        g_px.write64 = (write_value64_fn)fn;
    (void)cudaGetLastError();

    ishmemi_proxy_t &h = g_px.h_proxy;
    h.ring = g_px.ring;
    h.ring_slots = PROXY_RING_SLOTS;
    h.comp_slots = PROXY_COMP_SLOTS;
    h.head = g_px.d_words + 0;
    h.tail_cache = g_px.d_words + 1;
    h.comp_alloc = g_px.d_words + 2;
    h.nbi_issued = g_px.d_words + 8;
    h.nbi_seen = g_px.d_words + 8 + ISHMEM_MAX_PES;
    h.tail_pub = g_px.tail_pub;
    h.comp = g_px.comp;
    h.nbi_done = g_px.nbi_done;
    h.wg_cutover = g.wg_cutover;
    h.hybrid_head = g.hybrid_head;
    rc = ishmemi_cuda(cudaMemcpy(g_px.d_proxy, &h, sizeof(h), cudaMemcpyHostToDevice), "cudaMemcpy(proxy)");
    if (rc) {
        proxy_release();
        return rc;
    }
    g_px.stop.store(false);
    g_px.error.store(0);
    g_px.served.store(0);
    g_px.copies.store(0);
    g_px.thread = std::thread(proxy_main, g.device);
    g_px.running = true;
    for (int p = 0; p < g.npes; ++p) g.h_ctx[p].proxy = g_px.d_proxy;
    ishmemi_push_ctx();
    return ISHMEM_OK;
}

extern "C" int ishmemx_proxy_stop(void)
{
    ISHMEMI_REQUIRE_INIT();
    auto &g = g_ishmem;
    if (!g_px.running) return ISHMEM_OK;
    cudaDeviceSynchronize(); /* no kernel may still be posting */
    for (int p = 0; p < g.npes; ++p) g.h_ctx[p].proxy = nullptr;
    ishmemi_push_ctx();
    g_px.stop.store(true, std::memory_order_release);
    g_px.thread.join();
    cudaDeviceSynchronize(); /* replies still queued on the engine streams */
    g_px.running = false;
    proxy_release();
    return g_px.error.load() ? ISHMEM_ERR_CUDA : ISHMEM_OK;
}

void ishmemi_proxy_finalize()
{
    if (g_px.running) ishmemx_proxy_stop();
}

void ishmemi_proxy_set_cutover(size_t nbytes, size_t hybrid_head)
{
    if (!g_px.running) return;
    cudaDeviceSynchronize();
    g_px.h_proxy.wg_cutover = nbytes;
    g_px.h_proxy.hybrid_head = hybrid_head;
    cudaMemcpy(g_px.d_proxy, &g_px.h_proxy, sizeof(g_px.h_proxy), cudaMemcpyHostToDevice);
}

extern "C" int ishmemx_proxy_stats(uint64_t *requests_served, uint64_t *copies_started, int *uses_stream_memops)
{
    ISHMEMI_REQUIRE_INIT();
    if (requests_served) *requests_served = g_px.served.load();
    if (copies_started) *copies_started = g_px.copies.load();
    if (uses_stream_memops) *uses_stream_memops = g_px.write64 ? 1 : 0;
    return g_px.running ? ISHMEM_OK : ISHMEM_ERR_ARG;
}

/* ---- ring benchmark: round trip and request rate ------------------------------------------------ */

struct ring_bench_out {
    unsigned long long rtt_ns_sum, rtt_count, span_ns, posted, errors;
};
static_assert(sizeof(ring_bench_out) <= 64, "fits the 8 words reserved for it");

/* mode 0: every participating thread posts `iters` no-op requests one after another and waits
 * for each reply (round-trip time).  mode 1: every thread posts `iters` no-op requests without
 * reply, the last one with a reply (request rate as seen from the GPU). */
__global__ void __launch_bounds__(1024) k_ring_bench(const ishmem_ctx_t *ctxs, int mode, int iters, ring_bench_out *out)
{
    const ishmem_ctx_t *ctx = ctxs + (blockIdx.x % (unsigned)ctxs[0].npes);
    const ishmemi_proxy_t *px = ctx->proxy;
    if (px == nullptr) return;
    unsigned long long sum = 0, n = 0, err = 0;
    const unsigned long long t_begin = ishmemi::globaltimer_ns();
    for (int i = 0; i < iters; ++i) {
        const bool reply = (mode == 0) || (i == iters - 1);
        if (reply) {
            const unsigned long long c = atomicAdd(px->comp_alloc, 1ull);
            const unsigned long long t0 = ishmemi::globaltimer_ns();
            int rc = ishmemi::proxy_post(ctx, ISHMEMI_REQ_NOP, nullptr, nullptr, 0, nullptr, 0, c + 1);
            if (!rc) rc = ishmemi::proxy_wait(ctx, c);
            if (rc) {
                ++err;
                break;
            }
            sum += ishmemi::globaltimer_ns() - t0;
            ++n;
        } else if (ishmemi::proxy_post(ctx, ISHMEMI_REQ_NOP, nullptr, nullptr, 0, nullptr, 0, 0)) {
            ++err;
            break;
        }
    }
    const unsigned long long span = ishmemi::globaltimer_ns() - t_begin;
    atomicAdd(&out->rtt_ns_sum, sum);
    atomicAdd(&out->rtt_count, n);
    atomicMax(&out->span_ns, span);
    atomicAdd(&out->posted, (unsigned long long)iters);
    if (err) atomicAdd(&out->errors, err);
}

extern "C" int ishmemx_ring_benchmark(int mode, int blocks, int threads, int iters, double *mean_rtt_ns,
                                      double *requests_per_second)
{
    ISHMEMI_REQUIRE_INIT();
    auto &g = g_ishmem;
    if (!g_px.running) return ISHMEM_ERR_ARG;
    if (mode < 0 || mode > 1 || blocks < 1 || threads < 1 || threads > 1024 || iters < 1) return ISHMEM_ERR_ARG;
    ring_bench_out *d_out = (ring_bench_out *)(g_px.d_words + 8 + 2 * ISHMEM_MAX_PES);
    cudaStream_t s;
    int rc = ishmemi_team_stream_begin(ISHMEM_TEAM_WORLD, &s);
    if (rc) return rc;
    rc = ishmemi_cuda(cudaMemsetAsync(d_out, 0, sizeof(ring_bench_out), s), "cudaMemsetAsync");
    if (!rc) {
        k_ring_bench<<<blocks, threads, 0, s>>>(g.d_ctx, mode, iters, d_out);
        ishmemi_count_launch();
        rc = ishmemi_check_launch("k_ring_bench");
    }
    ishmemi_team_stream_end();
    if (rc) return rc;
    ISHMEMI_CUDA(cudaStreamSynchronize(s));
    ring_bench_out out;
    ISHMEMI_CUDA(cudaMemcpy(&out, d_out, sizeof(out), cudaMemcpyDeviceToHost));
    if (out.errors) return ISHMEM_ERR_TIMEOUT;
    if (mean_rtt_ns) *mean_rtt_ns = out.rtt_count ? (double)out.rtt_ns_sum / (double)out.rtt_count : 0.0;
    if (requests_per_second) *requests_per_second = out.span_ns ? (double)out.posted * 1e9 / (double)out.span_ns : 0.0;
    return ISHMEM_OK;
}
