/*
 * ishmem_device.cuh -- device-callable (GPU-initiated) part of the library, header only.
 *
 * Every routine takes the calling PE's context first (ishmemx_ctx(pe) on the host gives
 * the pointer).  Addresses follow OpenSHMEM: a symmetric object is named by its address
 * in the CALLING PE's own heap slice; the routine translates it to the target PE with
 * `addr - local_heap_base + remote_heap_base` after looking the PE up in the
 * reachable-by-store table (Section 3.3 last paragraph and Section 3.7.1 of the paper).
 *
 * Thread collaboration (Section 3.6): plain names are called by ONE thread (work-item);
 * *_sub_group by all 32 lanes of a converged warp; *_work_group by every thread of the
 * block, with the same arguments (they contain block-wide barriers).
 *
 * Written for sm_100a: 16-byte vector loads/stores, TMA bulk copies (cp.async.bulk) with
 * mbarrier staging for large aligned blocks, release/acquire at .gpu scope for signals,
 * and bounded waits everywhere (a wait that gives up latches ISHMEM_ERR_TIMEOUT in the
 * shared status word and returns that code; nothing here can spin forever).
 */
#ifndef ISHMEM_DEVICE_CUH
#define ISHMEM_DEVICE_CUH

#include <cuda_runtime.h>
#include <stdint.h>

#include "ishmem.h"

/* bytes of internal (non-heap) state per PE: sync counters and epochs per team */
#define ISHMEMI_INTERNAL_BYTES 1024

struct ishmemi_team {
    int start, stride, size, valid;
};

/* Reverse-offload request (Section 3.4 of the paper, "Synchronization with Host"): a fixed
 * 64-byte message that a GPU thread composes in a ring in host memory for the host proxy
 * thread.  `seq` (ticket + 1) is stored last, with release semantics at system scope: a slot
 * whose seq matches the host's expectation is complete. */
struct __align__(64) ishmemi_request {
    unsigned long long dest;       /* device address on the target PE (already translated) */
    unsigned long long src;        /* device address of the source */
    unsigned long long nbytes;
    unsigned long long sig_addr;   /* translated signal word, or 0 */
    unsigned long long sig_value;
    unsigned op;                   /* ISHMEMI_REQ_* */
    unsigned pe;                   /* issuing PE: selects the copy-engine stream */
    unsigned long long completion; /* completion ticket + 1, or 0: counted in nbi_done[pe] instead */
    unsigned long long seq;
};
#define ISHMEMI_REQ_NOP 0u        /* reply only (round-trip measurement) */
#define ISHMEMI_REQ_COPY 1u       /* cudaMemcpyAsync dest <- src on the issuing PE's engine stream */
#define ISHMEMI_REQ_COPY_SIGNAL 2u /* copy, then set the signal word, in stream order */

/* Device-side view of the ring.  The ring, the published tail and the completion words live in
 * pinned host memory mapped into the device's address space; the ticket counters live in device
 * memory.  Both directions use stores only; the GPU end needs no progress thread. */
struct ishmemi_proxy_t {
    ishmemi_request *ring;                 /* host memory, ring_slots entries */
    unsigned ring_slots;                   /* power of two */
    unsigned comp_slots;                   /* power of two */
    unsigned long long *head;              /* device: next ticket (one fetch-and-increment per message) */
    unsigned long long *tail_cache;        /* device: last value of *tail_pub any thread has seen */
    const unsigned long long *tail_pub;    /* host: messages consumed, published by the proxy now and then */
    unsigned long long *comp_alloc;        /* device: next completion ticket */
    const unsigned long long *comp;        /* host: slot c % comp_slots holds c + 1 once ticket c is complete */
    unsigned long long *nbi_issued;        /* device [npes]: non-blocking requests posted by each PE */
    unsigned long long *nbi_seen;          /* device [npes]: last value of nbi_done[pe] any thread has seen */
    const unsigned long long *nbi_done;    /* host [npes]: non-blocking requests of each PE completed */
    unsigned long long wg_cutover;         /* work-group put/get of at least this size use the engine */
    unsigned long long hybrid_head;        /* bytes the work-group copies itself while the engine starts on the rest */
};

/* Per-PE context, resident in device memory (Section 3.7.1: a separate GPU-side copy of
 * the runtime state, so that device calls never touch host memory). */
struct __align__(16) ishmem_ctx_t {
    int my_pe;
    int npes;
    unsigned long long heap_bytes;
    char *heap_base; /* this PE's slice */
    /* reach[pe] == 0: PE not reachable by load/store; otherwise heap_delta[pe] is the offset
     * between this PE's heap base and PE pe's heap base.  Both tables are indexed by the PE, so
     * that a translation is three independent loads (npes, flag, offset) and costs one trip to
     * the cache instead of a chain of them: after an acquire -- which every wait ends with -- none
     * of these hit in L1, and a chained look-up was half of a small put's latency. */
    unsigned char reach[ISHMEM_MAX_PES];
    long long heap_delta[ISHMEM_MAX_PES];
    /* internal region of this PE (outside the user heap): sync_arrive[team] is pushed by
     * the other members, sync_epoch[team] counts the syncs this PE has begun */
    unsigned long long *sync_arrive;
    unsigned long long *sync_epoch;
    unsigned long long *collect_sizes; /* [ISHMEM_MAX_PES]: contributions announced by the members of a collect */
    long long internal_stride; /* bytes between consecutive PEs' internal regions */
    ishmemi_team teams[ISHMEM_MAX_TEAMS];
    int *status;                       /* one word shared by all PEs; first error wins */
    unsigned long long wait_limit_ns;  /* time bound of every device-side wait */
    int bcast_root_dest;               /* broadcast writes the root's own dest */
    const ishmemi_proxy_t *proxy;      /* reverse-offload ring, or nullptr while no host proxy runs */
};

/* shared-memory staging handed to the *_work_group copy routines to enable the TMA bulk
 * path; {nullptr, 0} (the default) means loads/stores only */
struct ishmemx_staging_t {
    void *smem;          /* 128-byte aligned shared memory */
    unsigned bytes;      /* its size; at least 2 stages of 1 KiB plus 128 B are needed */
};

namespace ishmemi {

__device__ __forceinline__ void latch_error(const ishmem_ctx_t *ctx, int code)
{
    atomicCAS(ctx->status, 0, code);
}

__device__ __forceinline__ unsigned long long globaltimer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
/* Time bound of a spin loop: the first polls are free, after that the global timer is read
 * once per poll and compared with the limit. */
struct deadline {
    unsigned long long t0, limit_ns;
    unsigned polls;
    __device__ __forceinline__ explicit deadline(unsigned long long lim) : t0(0), limit_ns(lim), polls(0) {}
    __device__ __forceinline__ bool expired()
    {
        if (++polls < 128u) return false;
        const unsigned long long now = globaltimer_ns();
        if (t0 == 0) {
            t0 = now;
            return false;
        }
        return now - t0 > limit_ns;
    }
};

/* ---- address translation ------------------------------------------------------- */

/* Section 3.7.1: table lookup, load of the offset, pointer arithmetic.  Returns nullptr
 * (and latches an error) when pe is out of range or not reachable.  The three loads do not
 * depend on one another (the index is masked so that the tables can be read before the range
 * check is known). */
template <typename T>
__device__ __forceinline__ T *translate(const ishmem_ctx_t *ctx, const T *local_sym, int pe)
{
    const unsigned idx = (unsigned)pe & (ISHMEM_MAX_PES - 1);
    const int npes = ctx->npes;
    const unsigned reachable = ctx->reach[idx];
    const long long delta = ctx->heap_delta[idx];
    if ((unsigned)pe >= (unsigned)npes || reachable == 0) {
        latch_error(ctx, ISHMEM_ERR_INVALID_PE);
        return nullptr;
    }
    return (T *)((char *)local_sym + delta);
}

/* ---- memory-model primitives ---------------------------------------------------- */

__device__ __forceinline__ unsigned long long ld_acquire(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long ld_relaxed(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned ld_relaxed(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(unsigned long long *p, unsigned long long v)
{
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void st_relaxed(unsigned long long *p, unsigned long long v)
{
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void st_relaxed(unsigned *p, unsigned v)
{
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_release_add(unsigned long long *p, unsigned long long v)
{
    asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void fence_acq_rel_gpu()
{
    asm volatile("fence.acq_rel.gpu;" ::: "memory");
}
/* orders this thread's earlier generic-proxy accesses against later async-proxy (TMA)
 * accesses and vice versa */
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async;" ::: "memory");
}

/* ---- vector loads / stores -------------------------------------------------------- */

__device__ __forceinline__ uint4 ld16(const void *p)
{
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p)
                 : "memory");
    return v;
}
__device__ __forceinline__ void st16(void *p, uint4 v)
{
    asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
                 "r"(v.w)
                 : "memory");
}
template <typename V>
__device__ __forceinline__ V ldv(const void *p)
{
    return *(const volatile V *)p;
}
template <typename V>
__device__ __forceinline__ void stv(void *p, V v)
{
    *(volatile V *)p = v;
}

/* Copy with W-byte accesses, W in {1,2,4,8}; d, s and n multiples of W. */
template <typename V>
__device__ __forceinline__ void copy_words(char *d, const char *s, size_t n, unsigned tid,
                                           unsigned nthr)
{
    size_t nw = n / sizeof(V);
    size_t i = tid;
    for (; i + 3 * (size_t)nthr < nw; i += 4 * (size_t)nthr) {
        V a = ldv<V>(s + i * sizeof(V));
        V b = ldv<V>(s + (i + nthr) * sizeof(V));
        V c = ldv<V>(s + (i + 2 * (size_t)nthr) * sizeof(V));
        V e = ldv<V>(s + (i + 3 * (size_t)nthr) * sizeof(V));
        stv<V>(d + i * sizeof(V), a);
        stv<V>(d + (i + nthr) * sizeof(V), b);
        stv<V>(d + (i + 2 * (size_t)nthr) * sizeof(V), c);
        stv<V>(d + (i + 3 * (size_t)nthr) * sizeof(V), e);
    }
    for (; i < nw; i += nthr) stv<V>(d + i * sizeof(V), ldv<V>(s + i * sizeof(V)));
}

/* Body of a copy whose two addresses are congruent mod 16 and 16-byte aligned: `nvec`
 * 16-byte vectors, thread `tid` of `nthr` takes vectors tid, tid+nthr, ...; UNROLL
 * independent loads are issued before the first store. */
/* Groups of up to 512 threads also ask L2, two rounds ahead, for the lines they will load (one lane
 * per 128-byte line): the UNROLL vectors a thread holds in flight do not cover the DRAM latency of a
 * small group streaming a long message.  Measured on B200, 256 MiB: one group of 256 threads 53 -> 64
 * GB/s, 74 resident groups of 256 threads 2.9 -> 4.2 TB/s, 148 of them 4.4 -> 6.0 TB/s; groups of 1024
 * threads have enough in flight and lose a few per cent to the extra requests, so they do not
 * prefetch.  Messages of one or two rounds (the tiled launches) never reach a prefetch. */
#ifndef ISHMEMI_COPY_AHEAD
#define ISHMEMI_COPY_AHEAD 2
#endif
template <int UNROLL>
__device__ __forceinline__ void copy_vec16(char *d, const char *s, size_t nvec, unsigned tid,
                                           unsigned nthr)
{
    size_t i = tid;
    const size_t step = (size_t)nthr * UNROLL;
    const bool ahead = ISHMEMI_COPY_AHEAD > 0 && nthr <= 512u && (tid & 7u) == 0;
    for (; i + (size_t)(UNROLL - 1) * nthr < nvec; i += step) {
        if (ahead) {
#pragma unroll
            for (int k = 0; k < UNROLL; ++k) {
                const size_t j = i + (size_t)ISHMEMI_COPY_AHEAD * step + (size_t)k * nthr;
                if (j < nvec) asm volatile("prefetch.global.L2 [%0];" ::"l"(s + j * 16));
            }
        }
        uint4 v[UNROLL];
#pragma unroll
        for (int k = 0; k < UNROLL; ++k) v[k] = ld16(s + (i + (size_t)k * nthr) * 16);
#pragma unroll
        for (int k = 0; k < UNROLL; ++k) st16(d + (i + (size_t)k * nthr) * 16, v[k]);
    }
    for (; i < nvec; i += nthr) st16(d + i * 16, ld16(s + i * 16));
}

/* Fewer than 16 bytes at the edge of a vector copy: d and s are congruent mod 16, so the widest
 * power-of-two word that d is aligned to and that still fits is valid for both; at most
 * 1 + 2 + 4 + 8 bytes going up to a boundary or 8 + 4 + 2 + 1 coming down from one.  One thread. */
__device__ __forceinline__ void copy_edge(char *d, const char *s, size_t n)
{
    while (n) {
        const unsigned a = (unsigned)(uintptr_t)d;
        if (n >= 8 && (a & 7u) == 0) {
            stv<unsigned long long>(d, ldv<unsigned long long>(s));
            d += 8, s += 8, n -= 8;
        } else if (n >= 4 && (a & 3u) == 0) {
            stv<unsigned>(d, ldv<unsigned>(s));
            d += 4, s += 4, n -= 4;
        } else if (n >= 2 && (a & 1u) == 0) {
            stv<unsigned short>(d, ldv<unsigned short>(s));
            d += 2, s += 2, n -= 2;
        } else {
            stv<unsigned char>(d, ldv<unsigned char>(s));
            d += 1, s += 1, n -= 1;
        }
    }
}

/* General copy by `nthr` cooperating threads (nthr = 1: a single work-item).  Picks the
 * widest access both addresses allow: when dest and src are congruent mod 16 the head is
 * peeled to a 16-byte boundary and the body moves 16-byte vectors; otherwise the widest
 * power of two dividing their distance is used.  No synchronisation inside. */
template <int UNROLL = 4>
__device__ __forceinline__ void copy_bytes(char *d, const char *s, size_t n, unsigned tid,
                                           unsigned nthr)
{
    if (n == 0) return;
    const unsigned rel = (unsigned)((uintptr_t)d - (uintptr_t)s) & 15u;
    if (rel == 0) {
        size_t head = (size_t)((16u - ((unsigned)(uintptr_t)d & 15u)) & 15u);
        if (head > n) head = n;
        const size_t nvec = (n - head) >> 4, tail = n - head - (nvec << 4);
        /* the two ragged edges go to the first and the last thread, in the widest words */
        if (tid == 0) copy_edge(d, s, head);
        if (tid == nthr - 1) copy_edge(d + head + (nvec << 4), s + head + (nvec << 4), tail);
        copy_vec16<UNROLL>(d + head, s + head, nvec, tid, nthr);
        return;
    }
    /* W = widest power of two (< 16) dividing the distance between the two addresses */
    const unsigned W = rel & (0u - rel);
    size_t head = (size_t)((W - ((unsigned)(uintptr_t)d & (W - 1))) & (W - 1));
    if (head > n) head = n;
    for (size_t i = tid; i < head; i += nthr) stv<unsigned char>(d + i, ldv<unsigned char>(s + i));
    d += head;
    s += head;
    n -= head;
    const size_t body = n & ~(size_t)(W - 1);
    if (W == 8) copy_words<unsigned long long>(d, s, body, tid, nthr);
    else if (W == 4) copy_words<unsigned>(d, s, body, tid, nthr);
    else if (W == 2) copy_words<unsigned short>(d, s, body, tid, nthr);
    else copy_words<unsigned char>(d, s, body, tid, nthr);
    for (size_t i = body + tid; i < n; i += nthr) stv<unsigned char>(d + i, ldv<unsigned char>(s + i));
}

/* Strided element copy (iput / iget, the strided forms of Section 3.7.1): element k, taken every
 * `sst` elements from s, goes to element k*dst of d, k = tid, tid+nthr, ...  ES = element size in
 * bytes (1, 2, 4, 8 or 16); both addresses aligned to it. */
template <int ES>
struct strided_word;
template <> struct strided_word<1> { typedef unsigned char type; };
template <> struct strided_word<2> { typedef unsigned short type; };
template <> struct strided_word<4> { typedef unsigned type; };
template <> struct strided_word<8> { typedef unsigned long long type; };
template <> struct strided_word<16> { typedef uint4 type; };
template <int ES>
__device__ __forceinline__ typename strided_word<ES>::type strided_ld(const char *p)
{
    return ldv<typename strided_word<ES>::type>(p);
}
template <>
__device__ __forceinline__ uint4 strided_ld<16>(const char *p) { return ld16(p); }
template <int ES>
__device__ __forceinline__ void strided_st(char *p, typename strided_word<ES>::type v)
{
    stv<typename strided_word<ES>::type>(p, v);
}
template <>
__device__ __forceinline__ void strided_st<16>(char *p, uint4 v) { st16(p, v); }

/* elements tid, tid + nthr, ... of [0, nelems): four independent loads are in flight per thread
 * before the first store */
template <int ES>
__device__ __forceinline__ void strided_copy(char *d, const char *s, size_t dst, size_t sst, size_t nelems,
                                             size_t tid, size_t nthr)
{
    typedef typename strided_word<ES>::type W;
    size_t k = tid;
    for (; k + 3 * nthr < nelems; k += 4 * nthr) {
        W v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = strided_ld<ES>(s + (k + u * nthr) * sst * ES);
#pragma unroll
        for (int u = 0; u < 4; ++u) strided_st<ES>(d + (k + u * nthr) * dst * ES, v[u]);
    }
    for (; k < nelems; k += nthr) strided_st<ES>(d + k * dst * ES, strided_ld<ES>(s + k * sst * ES));
}
__device__ __forceinline__ void strided_copy_any(char *d, const char *s, size_t dst, size_t sst, size_t nelems,
                                                 unsigned es, size_t tid, size_t nthr)
{
    switch (es) {
    case 1: strided_copy<1>(d, s, dst, sst, nelems, tid, nthr); break;
    case 2: strided_copy<2>(d, s, dst, sst, nelems, tid, nthr); break;
    case 4: strided_copy<4>(d, s, dst, sst, nelems, tid, nthr); break;
    case 8: strided_copy<8>(d, s, dst, sst, nelems, tid, nthr); break;
    default: strided_copy<16>(d, s, dst, sst, nelems, tid, nthr); break;
    }
}

/* ---- TMA bulk copy ring --------------------------------------------------------------- */

__device__ __forceinline__ unsigned smem_u32(const void *p)
{
    return (unsigned)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_inval(unsigned bar)
{
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity)
{
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
/* bounded wait on one phase of an mbarrier */
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, unsigned long long limit_ns)
{
    deadline dl(limit_ns);
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (dl.expired()) return false;
    }
}
__device__ __forceinline__ void bulk_g2s(unsigned smem_dst, const void *gsrc, unsigned bytes,
                                         unsigned bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
            "r"(smem_dst),
        "l"(gsrc), "r"(bytes), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void bulk_s2g(void *gdst, unsigned smem_src, unsigned bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst),
                 "r"(smem_src), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit()
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait()
{
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}

#define ISHMEMI_MAX_STAGES 8

/* One thread streams `n` bytes (multiple of 16; d and s 16-byte aligned) through a ring of
 * shared-memory stages: global -> shared by cp.async.bulk completing on an mbarrier,
 * shared -> global by cp.async.bulk in bulk groups.  nstages-1 loads are kept in flight.
 * When `complete` is false the last stores may still be in flight on return (the _nbi
 * forms; ishmem_quiet by the same thread completes them) -- their shared-memory reads
 * are finished either way, so the staging may be reused.  With `delta` every staged chunk is
 * stored to the ndst destinations d + delta[q] (q != skip): the push form used by broadcast
 * and fcollect, one load and ndst stores per chunk.  Returns 0 or ISHMEM_ERR_TIMEOUT. */
static __device__ __noinline__ int bulk_copy_ring(const ishmem_ctx_t *ctx, char *d, const char *s,
                                                  size_t n, ishmemx_staging_t st, bool complete,
                                                  const long long *delta = nullptr, int ndst = 1,
                                                  int skip = -1, size_t first = 0, size_t stride = 1)
{
    /* layout: [0,64) mbarriers, [128, ...) stages */
    unsigned long long *bars = (unsigned long long *)st.smem;
    char *stage0 = (char *)st.smem + 128;
    unsigned avail = st.bytes - 128;
    unsigned nstages = ISHMEMI_MAX_STAGES;
    unsigned stage_bytes = (avail / nstages) & ~1023u;
    while (nstages > 2 && stage_bytes < 8192u) { /* prefer >= 8 KiB stages */
        --nstages;
        stage_bytes = (avail / nstages) & ~1023u;
    }
    if (stage_bytes > 65536u) stage_bytes = 65536u;
    /* chunks first, first + stride, ... of the range belong to this caller (blocks of one
     * launch take chunks round-robin so that together they sweep one contiguous window) */
    const size_t total = (n + stage_bytes - 1) / stage_bytes;
    const size_t nchunks = total > first ? (total - first + stride - 1) / stride : 0;
    const unsigned bar0 = smem_u32(bars);
    const unsigned sm0 = smem_u32(stage0);
    for (unsigned k = 0; k < nstages; ++k) mbar_init(bar0 + 8 * k, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();

    auto chunk_off = [&](size_t c) -> size_t { return (first + c * stride) * stage_bytes; };
    auto chunk_bytes = [&](size_t c) -> unsigned {
        size_t left = n - chunk_off(c);
        return left < stage_bytes ? (unsigned)left : stage_bytes;
    };
    auto issue_load = [&](size_t c) {
        unsigned sidx = (unsigned)(c % nstages);
        unsigned b = chunk_bytes(c);
        mbar_expect_tx(bar0 + 8 * sidx, b);
        bulk_g2s(sm0 + sidx * stage_bytes, s + chunk_off(c), b, bar0 + 8 * sidx);
    };

    int rc = 0;
    size_t issued = 0;
    for (; issued < nchunks && issued + 1 < nstages; ++issued) issue_load(issued);
    size_t c = 0;
    for (; c < nchunks; ++c) {
        unsigned sidx = (unsigned)(c % nstages);
        unsigned parity = (unsigned)((c / nstages) & 1);
        if (!mbar_wait(bar0 + 8 * sidx, parity, ctx->wait_limit_ns)) {
            rc = ISHMEM_ERR_TIMEOUT;
            break;
        }
        if (delta == nullptr) {
            bulk_s2g(d + chunk_off(c), sm0 + sidx * stage_bytes, chunk_bytes(c));
        } else {
            for (int q = 0; q < ndst; ++q)
                if (q != skip) bulk_s2g(d + delta[q] + chunk_off(c), sm0 + sidx * stage_bytes, chunk_bytes(c));
        }
        bulk_commit();
        if (issued < nchunks) {
            /* the stage of chunk c-1 is the one chunk `issued` will land in: its store
             * must have finished reading shared memory */
            bulk_wait_read<1>();
            issue_load(issued);
            ++issued;
        }
    }
    if (rc) {
        /* give the loads still in flight a bounded chance to land before the staging is
         * released, then report */
        latch_error(ctx, rc);
        for (size_t k = c + 1; k < issued; ++k)
            mbar_wait(bar0 + 8 * (unsigned)(k % nstages), (unsigned)((k / nstages) & 1),
                      ctx->wait_limit_ns);
    }
    if (complete || rc) {
        bulk_wait<0>();
        fence_proxy_async();
    } else {
        bulk_wait_read<0>();
    }
    for (unsigned k = 0; k < nstages; ++k) mbar_inval(bar0 + 8 * k);
    return rc;
}

/* ---- reverse offload: requests to the host proxy ------------------------------------------- */

__device__ __forceinline__ unsigned long long ld_acquire_sys(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.acquire.sys.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_sys(unsigned long long *p, unsigned long long v)
{
    asm volatile("st.release.sys.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

/* Polls of host memory cross the bus: every waiter backs off from 200 ns to 6.4 us between
 * polls, so that many waiters cannot crowd out the requests themselves. */
struct host_poll_backoff {
    unsigned ns;
    __device__ __forceinline__ host_poll_backoff() : ns(200u) {}
    __device__ __forceinline__ void pause()
    {
        __nanosleep(ns);
        if (ns < 6400u) ns <<= 1;
    }
};

/* Posts one request: one fetch-and-increment allocates the slot, the message is written with
 * plain stores and published by the release store of its sequence number.  Flow control (the
 * host must have consumed the slot's previous message) is checked against a cached copy of the
 * host's tail in device memory; host memory is only read when the ring looks full.  One thread
 * calls.  Returns 0 or ISHMEM_ERR_TIMEOUT. */
__device__ __forceinline__ int proxy_post(const ishmem_ctx_t *ctx, unsigned op, void *dest, const void *src,
                                          unsigned long long nbytes, unsigned long long *sig_addr,
                                          unsigned long long sig_value, unsigned long long completion)
{
    const ishmemi_proxy_t *px = ctx->proxy;
    const unsigned long long t = atomicAdd(px->head, 1ull);
    if (t - ld_relaxed(px->tail_cache) >= px->ring_slots) {
        deadline dl(ctx->wait_limit_ns);
        host_poll_backoff bo;
        for (;;) {
            /* somebody else may have refreshed the cached tail meanwhile */
            if (t - ld_relaxed(px->tail_cache) < px->ring_slots) break;
            const unsigned long long tail = ld_acquire_sys(px->tail_pub);
            if (t - tail < px->ring_slots) {
                atomicMax(px->tail_cache, tail);
                break;
            }
            if (dl.expired()) {
                latch_error(ctx, ISHMEM_ERR_TIMEOUT);
                return ISHMEM_ERR_TIMEOUT; /* the slot stays unwritten: the proxy stops at it */
            }
            bo.pause();
        }
    }
    ishmemi_request *slot = px->ring + (t & (px->ring_slots - 1));
    uint4 *w = (uint4 *)slot;
    const unsigned long long d = (unsigned long long)dest, sa = (unsigned long long)src, sg = (unsigned long long)sig_addr;
    w[0] = make_uint4((unsigned)d, (unsigned)(d >> 32), (unsigned)sa, (unsigned)(sa >> 32));
    w[1] = make_uint4((unsigned)nbytes, (unsigned)(nbytes >> 32), (unsigned)sg, (unsigned)(sg >> 32));
    w[2] = make_uint4((unsigned)sig_value, (unsigned)(sig_value >> 32), op, (unsigned)ctx->my_pe);
    slot->completion = completion;
    st_release_sys(&slot->seq, t + 1);
    return 0;
}

/* Waits (bounded) until completion ticket c has been answered; acquires at system scope, so
 * data the copy engine wrote before the reply is visible afterwards. */
__device__ __forceinline__ int proxy_wait(const ishmem_ctx_t *ctx, unsigned long long c)
{
    const ishmemi_proxy_t *px = ctx->proxy;
    const unsigned long long *word = px->comp + (c & (px->comp_slots - 1));
    deadline dl(ctx->wait_limit_ns);
    host_poll_backoff bo;
    for (;;) {
        if (ld_acquire_sys(word) >= c + 1) return 0;
        if (dl.expired()) break;
        bo.pause();
    }
    latch_error(ctx, ISHMEM_ERR_TIMEOUT);
    return ISHMEM_ERR_TIMEOUT;
}

/* All non-blocking engine requests posted so far by the calling PE are complete. */
__device__ __forceinline__ int proxy_quiet(const ishmem_ctx_t *ctx)
{
    const ishmemi_proxy_t *px = ctx->proxy;
    if (px == nullptr) return 0;
    const unsigned long long want = ld_relaxed(px->nbi_issued + ctx->my_pe);
    if (ld_relaxed(px->nbi_seen + ctx->my_pe) >= want) return 0;
    deadline dl(ctx->wait_limit_ns);
    host_poll_backoff bo;
    for (;;) {
        const unsigned long long done = ld_acquire_sys(px->nbi_done + ctx->my_pe);
        if (done >= want) {
            atomicMax(px->nbi_seen + ctx->my_pe, done);
            return 0;
        }
        if (dl.expired()) break;
        bo.pause();
    }
    latch_error(ctx, ISHMEM_ERR_TIMEOUT);
    return ISHMEM_ERR_TIMEOUT;
}

/* One thread hands a copy to the copy engine through the host proxy.  blocking: waits for the
 * reply.  Otherwise the request is counted for the PE and ishmem_quiet completes it. */
__device__ __forceinline__ int proxy_copy(const ishmem_ctx_t *ctx, char *d, const char *s, size_t n, bool blocking,
                                          unsigned long long *sig = nullptr, unsigned long long sig_value = 0)
{
    const ishmemi_proxy_t *px = ctx->proxy;
    const unsigned op = sig ? ISHMEMI_REQ_COPY_SIGNAL : ISHMEMI_REQ_COPY;
    if (blocking) {
        const unsigned long long c = atomicAdd(px->comp_alloc, 1ull);
        int rc = proxy_post(ctx, op, d, s, n, sig, sig_value, c + 1);
        return rc ? rc : proxy_wait(ctx, c);
    }
    atomicAdd(px->nbi_issued + ctx->my_pe, 1ull);
    return proxy_post(ctx, op, d, s, n, sig, sig_value, 0);
}

/* smallest aligned body worth starting the TMA ring for */
#define ISHMEMI_BULK_MIN_BYTES 16384u

/* work-group copy: all threads call.  Uses the TMA ring for the 16-byte-aligned body when
 * staging is given, the two addresses are congruent mod 16 and the body is large. */
__device__ __forceinline__ int wg_copy(const ishmem_ctx_t *ctx, char *d, const char *s, size_t n,
                                       ishmemx_staging_t st, bool complete)
{
    const unsigned tid = threadIdx.x + blockDim.x * (threadIdx.y + blockDim.y * threadIdx.z);
    const unsigned nthr = blockDim.x * blockDim.y * blockDim.z;
    if (ctx->proxy != nullptr && n >= ctx->proxy->wg_cutover) {
        /* cutover (Sections 3.2 and 3.7.1): above the tuned size the group leader asks the host
         * to start the copy engine, after a group barrier that makes the source valid */
        __shared__ int rc_engine;
        __shared__ unsigned long long ticket;
        /* hybrid form (a refinement the paper sketches): the engine gets the tail of the message
         * and, while it starts up, the group moves the head by loads and stores */
        size_t head = ctx->proxy->hybrid_head < n ? (size_t)ctx->proxy->hybrid_head & ~(size_t)255 : 0;
        if (!complete) head = 0; /* the non-blocking form returns at once */
        __syncthreads();
        if (tid == 0) {
            if (head) {
                ticket = atomicAdd(ctx->proxy->comp_alloc, 1ull);
                rc_engine = proxy_post(ctx, ISHMEMI_REQ_COPY, d + head, s + head, n - head, nullptr, 0, ticket + 1);
            } else {
                rc_engine = proxy_copy(ctx, d, s, n, complete);
            }
        }
        if (head) {
            copy_bytes(d, s, head, tid, nthr);
            if (tid == 0 && rc_engine == 0) rc_engine = proxy_wait(ctx, ticket);
        }
        __syncthreads();
        return rc_engine;
    }
    const bool congruent = ((((uintptr_t)d - (uintptr_t)s) & 15u) == 0);
    if (st.smem != nullptr && st.bytes >= 128u + 2048u && congruent && n >= ISHMEMI_BULK_MIN_BYTES) {
        size_t head = (size_t)((16u - ((unsigned)(uintptr_t)d & 15u)) & 15u);
        size_t body = (n - head) & ~(size_t)15;
        size_t tail = n - head - body;
        /* edges by loads/stores */
        for (size_t i = tid; i < head; i += nthr) stv<unsigned char>(d + i, ldv<unsigned char>(s + i));
        for (size_t i = tid; i < tail; i += nthr)
            stv<unsigned char>(d + head + body + i, ldv<unsigned char>(s + head + body + i));
        /* the source may have been written by this block's threads: make those writes
         * visible to the async proxy before the leader starts the bulk loads */
        fence_proxy_async();
        __syncthreads();
        __shared__ int rc_sh;
        if (tid == 0)
            rc_sh = bulk_copy_ring(ctx, d + head, s + head, body, st, complete);
        __syncthreads();
        return rc_sh;
    }
    copy_bytes(d, s, n, tid, nthr);
    return 0;
}

__device__ __forceinline__ bool compare(unsigned long long v, int cmp, unsigned long long ref)
{
    switch (cmp) {
    case ISHMEM_CMP_EQ: return v == ref;
    case ISHMEM_CMP_NE: return v != ref;
    case ISHMEM_CMP_GT: return v > ref;
    case ISHMEM_CMP_GE: return v >= ref;
    case ISHMEM_CMP_LT: return v < ref;
    default: return v <= ref;
    }
}

__device__ __forceinline__ void signal_update(unsigned long long *sig, unsigned long long v,
                                              int sig_op)
{
    if (sig_op == ISHMEM_SIGNAL_ADD) red_release_add(sig, v);
    else st_release(sig, v);
}

__device__ __forceinline__ unsigned block_tid()
{
    return threadIdx.x + blockDim.x * (threadIdx.y + blockDim.y * threadIdx.z);
}
__device__ __forceinline__ unsigned block_nthr() { return blockDim.x * blockDim.y * blockDim.z; }

} /* namespace ishmemi */

/* =============================== public device API =================================== */

/* PE `pe`'s copy of the symmetric object `local_sym` (named by its address in the calling
 * PE's heap), usable by plain loads and stores; nullptr if unreachable. */
template <typename T>
__device__ __forceinline__ T *ishmem_ptr(const ishmem_ctx_t *ctx, const T *local_sym, int pe)
{
    return ishmemi::translate(ctx, local_sym, pe);
}
/* Copies the calling PE's context into shared memory (all threads of the block call; ends with a
 * block barrier) and returns the copy, which every routine of this header accepts in place of
 * the original.  Worth it for kernels that issue many small operations: a routine reads its
 * context for the address translation, and after an acquire -- every successful wait is one --
 * those reads miss L1 and go to L2, 170 to 420 ns per trip on B200 depending on the L2 partition
 * the context happens to live in; from shared memory they cost a few cycles.  The context does
 * not change while a kernel runs (the host rewrites it only between launches), and the pointers
 * inside it keep naming the same global state. */
__device__ __forceinline__ const ishmem_ctx_t *ishmemx_ctx_stage_work_group(ishmem_ctx_t *smem_ctx,
                                                                            const ishmem_ctx_t *ctx)
{
    static_assert(sizeof(ishmem_ctx_t) % 16 == 0, "copied in 16-byte words");
    const unsigned tid = ishmemi::block_tid(), nthr = ishmemi::block_nthr();
    for (unsigned i = tid; i < sizeof(ishmem_ctx_t) / 16; i += nthr) ((uint4 *)smem_ctx)[i] = ((const uint4 *)ctx)[i];
    __syncthreads();
    return smem_ctx;
}
__device__ __forceinline__ int ishmem_my_pe(const ishmem_ctx_t *ctx) { return ctx->my_pe; }
__device__ __forceinline__ int ishmem_n_pes(const ishmem_ctx_t *ctx) { return ctx->npes; }

/* ---- scalar p / g (Section 3.7.1, the ishmem_long_p example) ------------------------- */
template <typename T>
__device__ __forceinline__ void ishmem_p(const ishmem_ctx_t *ctx, T *dest, T value, int pe)
{
    T *r = ishmemi::translate(ctx, dest, pe);
    if (r) *(volatile T *)r = value;
}
template <typename T>
__device__ __forceinline__ T ishmem_g(const ishmem_ctx_t *ctx, const T *src, int pe)
{
    const T *r = ishmemi::translate(ctx, src, pe);
    return r ? *(const volatile T *)r : T();
}
__device__ __forceinline__ void ishmem_long_p(const ishmem_ctx_t *ctx, long *dest, long value, int pe)
{
    ishmem_p<long>(ctx, dest, value, pe);
}
__device__ __forceinline__ long ishmem_long_g(const ishmem_ctx_t *ctx, const long *src, int pe)
{
    return ishmem_g<long>(ctx, src, pe);
}

/* ---- block put / get ------------------------------------------------------------------ */

/* work-item: one thread runs the vectorised copy (Section 3.7.1). */
__device__ __forceinline__ void ishmem_putmem(const ishmem_ctx_t *ctx, void *dest, const void *src,
                                              size_t nbytes, int pe)
{
    char *r = ishmemi::translate(ctx, (char *)dest, pe);
    if (r) ishmemi::copy_bytes<8>(r, (const char *)src, nbytes, 0, 1);
}
__device__ __forceinline__ void ishmem_getmem(const ishmem_ctx_t *ctx, void *dest, const void *src,
                                              size_t nbytes, int pe)
{
    const char *r = ishmemi::translate(ctx, (const char *)src, pe);
    if (r) ishmemi::copy_bytes<8>((char *)dest, r, nbytes, 0, 1);
}
template <typename T>
__device__ __forceinline__ void ishmem_put(const ishmem_ctx_t *ctx, T *dest, const T *src,
                                           size_t nelems, int pe)
{
    ishmem_putmem(ctx, dest, src, nelems * sizeof(T), pe);
}
template <typename T>
__device__ __forceinline__ void ishmem_get(const ishmem_ctx_t *ctx, T *dest, const T *src,
                                           size_t nelems, int pe)
{
    ishmem_getmem(ctx, dest, src, nelems * sizeof(T), pe);
}
/* Non-blocking forms: loads and stores are already asynchronous to the issuing thread; the
 * data is guaranteed delivered after ishmem_quiet. */
__device__ __forceinline__ void ishmem_putmem_nbi(const ishmem_ctx_t *ctx, void *dest,
                                                  const void *src, size_t nbytes, int pe)
{
    ishmem_putmem(ctx, dest, src, nbytes, pe);
}
__device__ __forceinline__ void ishmem_getmem_nbi(const ishmem_ctx_t *ctx, void *dest,
                                                  const void *src, size_t nbytes, int pe)
{
    ishmem_getmem(ctx, dest, src, nbytes, pe);
}

/* sub-group: the 32 lanes of a converged warp share the copy. */
__device__ __forceinline__ void ishmemx_putmem_sub_group(const ishmem_ctx_t *ctx, void *dest,
                                                         const void *src, size_t nbytes, int pe)
{
    char *r = ishmemi::translate(ctx, (char *)dest, pe);
    if (r) ishmemi::copy_bytes(r, (const char *)src, nbytes, threadIdx.x & 31u, 32u);
    __syncwarp();
}
__device__ __forceinline__ void ishmemx_getmem_sub_group(const ishmem_ctx_t *ctx, void *dest,
                                                         const void *src, size_t nbytes, int pe)
{
    const char *r = ishmemi::translate(ctx, (const char *)src, pe);
    if (r) ishmemi::copy_bytes((char *)dest, r, nbytes, threadIdx.x & 31u, 32u);
    __syncwarp();
}

/* strided put / get (OpenSHMEM iput / iget): strides in elements, at least 1.  T of 1, 2, 4, 8
 * or 16 bytes.  The plain forms are called by one thread, the _work_group forms by every thread
 * of the block (they end with a block barrier). */
template <typename T>
__device__ __forceinline__ void ishmem_iput(const ishmem_ctx_t *ctx, T *dest, const T *src, size_t dst, size_t sst,
                                            size_t nelems, int pe)
{
    char *r = ishmemi::translate(ctx, (char *)dest, pe);
    if (r) ishmemi::strided_copy<sizeof(T)>(r, (const char *)src, dst, sst, nelems, 0, 1);
}
template <typename T>
__device__ __forceinline__ void ishmem_iget(const ishmem_ctx_t *ctx, T *dest, const T *src, size_t dst, size_t sst,
                                            size_t nelems, int pe)
{
    const char *r = ishmemi::translate(ctx, (const char *)src, pe);
    if (r) ishmemi::strided_copy<sizeof(T)>((char *)dest, r, dst, sst, nelems, 0, 1);
}
template <typename T>
__device__ __forceinline__ void ishmemx_iput_work_group(const ishmem_ctx_t *ctx, T *dest, const T *src, size_t dst,
                                                        size_t sst, size_t nelems, int pe)
{
    char *r = ishmemi::translate(ctx, (char *)dest, pe);
    if (r)
        ishmemi::strided_copy<sizeof(T)>(r, (const char *)src, dst, sst, nelems,
                                         threadIdx.x + blockDim.x * (threadIdx.y + blockDim.y * threadIdx.z),
                                         blockDim.x * blockDim.y * blockDim.z);
    __syncthreads();
}
template <typename T>
__device__ __forceinline__ void ishmemx_iget_work_group(const ishmem_ctx_t *ctx, T *dest, const T *src, size_t dst,
                                                        size_t sst, size_t nelems, int pe)
{
    const char *r = ishmemi::translate(ctx, (const char *)src, pe);
    if (r)
        ishmemi::strided_copy<sizeof(T)>((char *)dest, r, dst, sst, nelems,
                                         threadIdx.x + blockDim.x * (threadIdx.y + blockDim.y * threadIdx.z),
                                         blockDim.x * blockDim.y * blockDim.z);
    __syncthreads();
}

/* work-group: every thread of the block takes part in a multi-threaded vectorised copy
 * (Sections 3.6, 3.7.1); with `staging` large aligned blocks are moved by TMA bulk copies
 * instead.  Returns 0 or ISHMEM_ERR_TIMEOUT (same value in every thread).  On return the
 * source may be reused; the data is ordered before any later signal/sync by this block. */
__device__ __forceinline__ int ishmemx_putmem_work_group(const ishmem_ctx_t *ctx, void *dest,
                                                         const void *src, size_t nbytes, int pe,
                                                         ishmemx_staging_t staging = {nullptr, 0})
{
    char *r = ishmemi::translate(ctx, (char *)dest, pe);
    int rc = ISHMEM_ERR_INVALID_PE;
    if (r) rc = ishmemi::wg_copy(ctx, r, (const char *)src, nbytes, staging, true);
    __syncthreads();
    return rc;
}
__device__ __forceinline__ int ishmemx_getmem_work_group(const ishmem_ctx_t *ctx, void *dest,
                                                         const void *src, size_t nbytes, int pe,
                                                         ishmemx_staging_t staging = {nullptr, 0})
{
    const char *r = ishmemi::translate(ctx, (const char *)src, pe);
    int rc = ISHMEM_ERR_INVALID_PE;
    if (r) rc = ishmemi::wg_copy(ctx, (char *)dest, r, nbytes, staging, true);
    __syncthreads();
    return rc;
}
/* _nbi: returns once the copy is issued; with staging the last bulk stores may still be in
 * flight until ishmemx_quiet_work_group / ishmem_quiet. */
__device__ __forceinline__ int ishmemx_putmem_nbi_work_group(const ishmem_ctx_t *ctx, void *dest,
                                                             const void *src, size_t nbytes, int pe,
                                                             ishmemx_staging_t staging = {nullptr, 0})
{
    char *r = ishmemi::translate(ctx, (char *)dest, pe);
    int rc = ISHMEM_ERR_INVALID_PE;
    if (r) rc = ishmemi::wg_copy(ctx, r, (const char *)src, nbytes, staging, false);
    return rc;
}
__device__ __forceinline__ int ishmemx_getmem_nbi_work_group(const ishmem_ctx_t *ctx, void *dest,
                                                             const void *src, size_t nbytes, int pe,
                                                             ishmemx_staging_t staging = {nullptr, 0})
{
    const char *r = ishmemi::translate(ctx, (const char *)src, pe);
    int rc = ISHMEM_ERR_INVALID_PE;
    if (r) rc = ishmemi::wg_copy(ctx, (char *)dest, r, nbytes, staging, false);
    return rc;
}

/* Explicit copy-engine forms (device-initiated reverse offload, Sections 3.4 and 3.7.1): after a
 * group barrier the leader posts one request to the host proxy, which starts the engine; the
 * other threads are free until the closing barrier.  Need a running proxy (ishmemx_proxy_start),
 * else ISHMEM_ERR_ARG.  The blocking form returns when the data has arrived; the _nbi form when
 * the request is posted (ishmem_quiet / ishmemx_quiet_work_group complete it). */
__device__ __forceinline__ int ishmemx_putmem_engine_work_group(const ishmem_ctx_t *ctx, void *dest,
                                                                const void *src, size_t nbytes, int pe,
                                                                bool blocking = true)
{
    char *r = ishmemi::translate(ctx, (char *)dest, pe);
    __shared__ int rc_sh;
    __syncthreads();
    if (ishmemi::block_tid() == 0)
        rc_sh = !r ? ISHMEM_ERR_INVALID_PE
                   : (ctx->proxy == nullptr ? ISHMEM_ERR_ARG
                                            : (nbytes ? ishmemi::proxy_copy(ctx, r, (const char *)src, nbytes, blocking) : 0));
    __syncthreads();
    return rc_sh;
}
__device__ __forceinline__ int ishmemx_getmem_engine_work_group(const ishmem_ctx_t *ctx, void *dest,
                                                                const void *src, size_t nbytes, int pe,
                                                                bool blocking = true)
{
    const char *r = ishmemi::translate(ctx, (const char *)src, pe);
    __shared__ int rc_sh;
    __syncthreads();
    if (ishmemi::block_tid() == 0)
        rc_sh = !r ? ISHMEM_ERR_INVALID_PE
                   : (ctx->proxy == nullptr ? ISHMEM_ERR_ARG
                                            : (nbytes ? ishmemi::proxy_copy(ctx, (char *)dest, r, nbytes, blocking) : 0));
    __syncthreads();
    return rc_sh;
}
/* put through the engine followed by SIGNAL_SET of the signal word, both in the engine's stream
 * order; non-blocking (the waiter's wait_until on the signal is the completion). */
__device__ __forceinline__ int ishmemx_putmem_signal_engine_work_group(const ishmem_ctx_t *ctx, void *dest,
                                                                       const void *src, size_t nbytes,
                                                                       unsigned long long *sig_addr,
                                                                       unsigned long long signal, int pe)
{
    char *r = ishmemi::translate(ctx, (char *)dest, pe);
    unsigned long long *rs = ishmemi::translate(ctx, sig_addr, pe);
    __shared__ int rc_sh;
    __syncthreads();
    if (ishmemi::block_tid() == 0)
        rc_sh = (!r || !rs) ? ISHMEM_ERR_INVALID_PE
                            : (ctx->proxy == nullptr ? ISHMEM_ERR_ARG
                                                     : ishmemi::proxy_copy(ctx, r, (const char *)src, nbytes, false, rs, signal));
    __syncthreads();
    return rc_sh;
}

/* ---- ordering --------------------------------------------------------------------------- */

/* fence: this thread's earlier puts are ordered before its later puts and signals. */
__device__ __forceinline__ void ishmem_fence(const ishmem_ctx_t *) { ishmemi::fence_acq_rel_gpu(); }
/* quiet: all operations issued by this thread are complete and visible device-wide,
 * including bulk stores left in flight by _nbi calls and, for the calling PE, copies handed to
 * the copy engine by _nbi calls above the cutover (a timeout there is latched in the status
 * word). */
__device__ __forceinline__ void ishmem_quiet(const ishmem_ctx_t *ctx)
{
    ishmemi::bulk_wait<0>();
    ishmemi::fence_proxy_async();
    ishmemi::fence_acq_rel_gpu();
    if (ctx->proxy != nullptr) (void)ishmemi::proxy_quiet(ctx); /* requests left with the copy engine */
}
__device__ __forceinline__ void ishmemx_quiet_work_group(const ishmem_ctx_t *ctx)
{
    ishmemi::bulk_wait<0>();
    ishmemi::fence_proxy_async();
    ishmemi::fence_acq_rel_gpu();
    /* one thread waits for the copy engine on behalf of the group */
    if (ctx->proxy != nullptr && ishmemi::block_tid() == 0) (void)ishmemi::proxy_quiet(ctx);
    __syncthreads();
}

/* ---- signalling and point-to-point synchronisation -------------------------------------- */

__device__ __forceinline__ void ishmem_putmem_signal(const ishmem_ctx_t *ctx, void *dest,
                                                     const void *src, size_t nbytes,
                                                     unsigned long long *sig_addr,
                                                     unsigned long long signal, int sig_op, int pe)
{
    char *r = ishmemi::translate(ctx, (char *)dest, pe);
    unsigned long long *rs = ishmemi::translate(ctx, sig_addr, pe);
    if (!r || !rs) return;
    ishmemi::copy_bytes<8>(r, (const char *)src, nbytes, 0, 1);
    ishmemi::signal_update(rs, signal, sig_op); /* release: payload first */
}
/* All threads copy; after a block barrier the leader releases the signal word, so the
 * waiter that acquires it sees the whole payload.  Above the work-group cutover (host proxy
 * running, SIGNAL_SET) payload and signal go through the copy engine instead, in its stream
 * order, and the call returns once the request is posted. */
__device__ __forceinline__ int ishmemx_putmem_signal_work_group(
    const ishmem_ctx_t *ctx, void *dest, const void *src, size_t nbytes,
    unsigned long long *sig_addr, unsigned long long signal, int sig_op, int pe,
    ishmemx_staging_t staging = {nullptr, 0})
{
    if (ctx->proxy != nullptr && nbytes >= ctx->proxy->wg_cutover && sig_op == ISHMEM_SIGNAL_SET)
        return ishmemx_putmem_signal_engine_work_group(ctx, dest, src, nbytes, sig_addr, signal, pe);
    char *r = ishmemi::translate(ctx, (char *)dest, pe);
    unsigned long long *rs = ishmemi::translate(ctx, sig_addr, pe);
    int rc = ISHMEM_ERR_INVALID_PE;
    if (r && rs) rc = ishmemi::wg_copy(ctx, r, (const char *)src, nbytes, staging, true);
    __syncthreads();
    /* the release below is cumulative: it also covers the other threads' stores, which the
     * block barrier has ordered before it */
    /* no signal after a copy that gave up (rc is the same in every thread): the waiter must
     * never acquire a signal whose payload is incomplete */
    if (rc == 0 && ishmemi::block_tid() == 0) ishmemi::signal_update(rs, signal, sig_op);
    return rc;
}
__device__ __forceinline__ unsigned long long ishmem_signal_fetch(const ishmem_ctx_t *,
                                                                  const unsigned long long *sig_addr)
{
    return ishmemi::ld_acquire(sig_addr);
}

/* Bounded wait until (*ivar cmp value) on the calling PE's own copy.  Returns 0, or
 * ISHMEM_ERR_TIMEOUT after ctx->wait_limit_ns (also latched in the status word). */
__device__ __forceinline__ int ishmem_uint64_wait_until(const ishmem_ctx_t *ctx,
                                                        const unsigned long long *ivar, int cmp,
                                                        unsigned long long value)
{
    ishmemi::deadline dl(ctx->wait_limit_ns);
    for (;;) {
        if (ishmemi::compare(ishmemi::ld_acquire(ivar), cmp, value)) return 0;
        if (dl.expired()) break;
        if (dl.polls > 64u) __nanosleep(dl.polls > 4096u ? 256 : 32);
    }
    ishmemi::latch_error(ctx, ISHMEM_ERR_TIMEOUT);
    return ISHMEM_ERR_TIMEOUT;
}
__device__ __forceinline__ int ishmemx_uint64_wait_until_work_group(const ishmem_ctx_t *ctx,
                                                                    const unsigned long long *ivar,
                                                                    int cmp, unsigned long long value)
{
    __shared__ int rc_sh;
    if (ishmemi::block_tid() == 0) rc_sh = ishmem_uint64_wait_until(ctx, ivar, cmp, value);
    __syncthreads();
    int rc = rc_sh;
    __syncthreads();
    return rc;
}
/* one non-blocking evaluation of the condition */
__device__ __forceinline__ int ishmem_uint64_test(const ishmem_ctx_t *, const unsigned long long *ivar,
                                                  int cmp, unsigned long long value)
{
    return ishmemi::compare(ishmemi::ld_acquire(ivar), cmp, value) ? 1 : 0;
}

/* Waits on `nelems` consecutive 64-bit words of the calling PE (OpenSHMEM 1.5 wait_until_all /
 * _any / _some).  `status` (may be nullptr) is OpenSHMEM's mask: words whose status entry is
 * non-zero are left out of the wait.  One thread calls.  All three are bounded
 * by ctx->wait_limit_ns and return 0 or ISHMEM_ERR_TIMEOUT (latched).
 * _all: every word satisfies the comparison.
 * _any: *index = some word that does (the lowest one found in a scan from 0).
 * _some: waits until at least one does, then lists ALL that do at that moment in indices[]
 *        (ascending, room for nelems entries) and their number in *count. */
__device__ __forceinline__ int ishmem_uint64_wait_until_all(const ishmem_ctx_t *ctx, const unsigned long long *ivars,
                                                            size_t nelems, int cmp, unsigned long long value,
                                                            const int *status = nullptr)
{
    ishmemi::deadline dl(ctx->wait_limit_ns);
    size_t k = 0;
    while (k < nelems) {
        if ((status && status[k]) || ishmemi::compare(ishmemi::ld_acquire(ivars + k), cmp, value)) {
            ++k;
            continue;
        }
        if (dl.expired()) {
            ishmemi::latch_error(ctx, ISHMEM_ERR_TIMEOUT);
            return ISHMEM_ERR_TIMEOUT;
        }
        if (dl.polls > 64u) __nanosleep(32);
    }
    return 0;
}
__device__ __forceinline__ int ishmem_uint64_wait_until_any(const ishmem_ctx_t *ctx, const unsigned long long *ivars,
                                                            size_t nelems, int cmp, unsigned long long value,
                                                            size_t *index, const int *status = nullptr)
{
    ishmemi::deadline dl(ctx->wait_limit_ns);
    if (nelems == 0) return 0;
    for (;;) {
        for (size_t k = 0; k < nelems; ++k)
            if (!(status && status[k]) && ishmemi::compare(ishmemi::ld_acquire(ivars + k), cmp, value)) {
                *index = k;
                return 0;
            }
        if (dl.expired()) break;
        if (dl.polls > 64u) __nanosleep(32);
    }
    ishmemi::latch_error(ctx, ISHMEM_ERR_TIMEOUT);
    return ISHMEM_ERR_TIMEOUT;
}
__device__ __forceinline__ int ishmem_uint64_wait_until_some(const ishmem_ctx_t *ctx, const unsigned long long *ivars,
                                                             size_t nelems, size_t *indices, int cmp,
                                                             unsigned long long value, size_t *count,
                                                             const int *status = nullptr)
{
    ishmemi::deadline dl(ctx->wait_limit_ns);
    *count = 0;
    if (nelems == 0) return 0;
    for (;;) {
        size_t n = 0;
        for (size_t k = 0; k < nelems; ++k)
            if (!(status && status[k]) && ishmemi::compare(ishmemi::ld_acquire(ivars + k), cmp, value))
                indices[n++] = k;
        if (n) {
            *count = n;
            return 0;
        }
        if (dl.expired()) break;
        if (dl.polls > 64u) __nanosleep(32);
    }
    ishmemi::latch_error(ctx, ISHMEM_ERR_TIMEOUT);
    return ISHMEM_ERR_TIMEOUT;
}

/* ---- remote atomics (scalar: no work-group forms, Section 3.6) --------------------------- */
/* T in {int, unsigned, long long, unsigned long long, long, unsigned long, int32_t, ...}
 * of 4 or 8 bytes.  Relaxed at .gpu scope; ordering comes from fence / quiet. */
namespace ishmemi {
template <typename T, int S = sizeof(T)>
struct amo;
template <typename T>
struct amo<T, 4> {
    typedef unsigned U;
    static __device__ __forceinline__ T fetch_add(T *p, T v) { return (T)atomicAdd((U *)p, (U)v); }
    static __device__ __forceinline__ T swap(T *p, T v) { return (T)atomicExch((U *)p, (U)v); }
    static __device__ __forceinline__ T cas(T *p, T c, T v) { return (T)atomicCAS((U *)p, (U)c, (U)v); }
    static __device__ __forceinline__ T fetch_and(T *p, T v) { return (T)atomicAnd((U *)p, (U)v); }
    static __device__ __forceinline__ T fetch_or(T *p, T v) { return (T)atomicOr((U *)p, (U)v); }
    static __device__ __forceinline__ T fetch_xor(T *p, T v) { return (T)atomicXor((U *)p, (U)v); }
    static __device__ __forceinline__ T fetch(const T *p) { return (T)ld_relaxed((const U *)p); }
    static __device__ __forceinline__ void set(T *p, T v) { st_relaxed((U *)p, (U)v); }
};
template <typename T>
struct amo<T, 8> {
    typedef unsigned long long U;
    static __device__ __forceinline__ T fetch_add(T *p, T v) { return (T)atomicAdd((U *)p, (U)v); }
    static __device__ __forceinline__ T swap(T *p, T v) { return (T)atomicExch((U *)p, (U)v); }
    static __device__ __forceinline__ T cas(T *p, T c, T v) { return (T)atomicCAS((U *)p, (U)c, (U)v); }
    static __device__ __forceinline__ T fetch_and(T *p, T v) { return (T)atomicAnd((U *)p, (U)v); }
    static __device__ __forceinline__ T fetch_or(T *p, T v) { return (T)atomicOr((U *)p, (U)v); }
    static __device__ __forceinline__ T fetch_xor(T *p, T v) { return (T)atomicXor((U *)p, (U)v); }
    static __device__ __forceinline__ T fetch(const T *p) { return (T)ld_relaxed((const U *)p); }
    static __device__ __forceinline__ void set(T *p, T v) { st_relaxed((U *)p, (U)v); }
};
} /* namespace ishmemi */

#define ISHMEMI_AMO2(NAME, CALL)                                                                  \
    template <typename T>                                                                         \
    __device__ __forceinline__ T ishmem_atomic_##NAME(const ishmem_ctx_t *ctx, T *target, T value, \
                                                      int pe)                                     \
    {                                                                                             \
        T *r = ishmemi::translate(ctx, target, pe);                                               \
        return r ? ishmemi::amo<T>::CALL(r, value) : T();                                         \
    }
ISHMEMI_AMO2(fetch_add, fetch_add)
ISHMEMI_AMO2(swap, swap)
ISHMEMI_AMO2(fetch_and, fetch_and)
ISHMEMI_AMO2(fetch_or, fetch_or)
ISHMEMI_AMO2(fetch_xor, fetch_xor)
#undef ISHMEMI_AMO2
template <typename T>
__device__ __forceinline__ void ishmem_atomic_add(const ishmem_ctx_t *ctx, T *target, T value, int pe)
{
    T *r = ishmemi::translate(ctx, target, pe);
    if (r) (void)ishmemi::amo<T>::fetch_add(r, value); /* result unused: compiles to a reduction */
}
/* non-fetching bitwise forms: the result is unused, so each compiles to a reduction */
#define ISHMEMI_AMO_NF(NAME)                                                                          \
    template <typename T>                                                                             \
    __device__ __forceinline__ void ishmem_atomic_##NAME(const ishmem_ctx_t *ctx, T *target, T value, \
                                                         int pe)                                      \
    {                                                                                                 \
        T *r = ishmemi::translate(ctx, target, pe);                                                   \
        if (r) (void)ishmemi::amo<T>::fetch_##NAME(r, value);                                         \
    }
ISHMEMI_AMO_NF(and)
ISHMEMI_AMO_NF(or)
ISHMEMI_AMO_NF(xor)
#undef ISHMEMI_AMO_NF
template <typename T>
__device__ __forceinline__ T ishmem_atomic_fetch_inc(const ishmem_ctx_t *ctx, T *target, int pe)
{
    return ishmem_atomic_fetch_add<T>(ctx, target, (T)1, pe);
}
template <typename T>
__device__ __forceinline__ void ishmem_atomic_inc(const ishmem_ctx_t *ctx, T *target, int pe)
{
    ishmem_atomic_add<T>(ctx, target, (T)1, pe);
}
template <typename T>
__device__ __forceinline__ T ishmem_atomic_fetch(const ishmem_ctx_t *ctx, const T *target, int pe)
{
    const T *r = ishmemi::translate(ctx, target, pe);
    return r ? ishmemi::amo<T>::fetch(r) : T();
}
template <typename T>
__device__ __forceinline__ void ishmem_atomic_set(const ishmem_ctx_t *ctx, T *target, T value, int pe)
{
    T *r = ishmemi::translate(ctx, target, pe);
    if (r) ishmemi::amo<T>::set(r, value);
}
template <typename T>
__device__ __forceinline__ T ishmem_atomic_compare_swap(const ishmem_ctx_t *ctx, T *target, T cond,
                                                        T value, int pe)
{
    T *r = ishmemi::translate(ctx, target, pe);
    return r ? ishmemi::amo<T>::cas(r, cond, value) : T();
}

/* ---- sync / barrier (Section 3.7.2, "Sync and Broadcast") --------------------------------- */

/* Push synchronisation of a team, called by ONE work-group per member PE: every thread
 * sends fire-and-forget atomic increments to the other members' arrival counters (they
 * pipeline), then the leader polls this PE's own counter until it reaches
 * epoch * team_size.  Counters are monotone; nothing is ever reset.  Returns 0 or
 * ISHMEM_ERR_TIMEOUT in every thread. */
__device__ __forceinline__ int ishmemx_team_sync_work_group(const ishmem_ctx_t *ctx,
                                                            ishmem_team_t team)
{
    const ishmemi_team t = ctx->teams[team];
    const unsigned tid = ishmemi::block_tid(), nthr = ishmemi::block_nthr();
    __shared__ int rc_sh;
    __syncthreads(); /* this block's earlier stores precede the increments */
    for (unsigned i = tid; i < (unsigned)t.size; i += nthr) {
        int pe = t.start + (int)i * t.stride;
        unsigned long long *remote = (unsigned long long *)((char *)(ctx->sync_arrive + team) +
                                                            (long long)(pe - ctx->my_pe) *
                                                                ctx->internal_stride);
        ishmemi::red_release_add(remote, 1ull);
    }
    if (tid == 0) {
        unsigned long long epoch = ctx->sync_epoch[team] + 1;
        ctx->sync_epoch[team] = epoch;
        const unsigned long long want = epoch * (unsigned long long)t.size;
        ishmemi::deadline dl(ctx->wait_limit_ns);
        int rc = 0;
        while (ishmemi::ld_acquire(ctx->sync_arrive + team) < want) {
            if (dl.expired()) {
                rc = ISHMEM_ERR_TIMEOUT;
                break;
            }
            if (dl.polls > 64u) __nanosleep(32);
        }
        if (rc) ishmemi::latch_error(ctx, rc);
        rc_sh = rc;
    }
    __syncthreads();
    int rc = rc_sh;
    __syncthreads();
    return rc;
}
__device__ __forceinline__ int ishmemx_sync_all_work_group(const ishmem_ctx_t *ctx)
{
    return ishmemx_team_sync_work_group(ctx, ISHMEM_TEAM_WORLD);
}
/* barrier = quiet + sync */
__device__ __forceinline__ int ishmemx_barrier_all_work_group(const ishmem_ctx_t *ctx)
{
    ishmem_quiet(ctx);
    return ishmemx_team_sync_work_group(ctx, ISHMEM_TEAM_WORLD);
}

/* ---- collectives (Section 3.7.2) ------------------------------------------------------------ */

namespace ishmemi {

template <typename T, int OP>
__device__ __forceinline__ T combine(T acc, T x)
{
    if (OP == ISHMEM_OP_SUM) return acc + x;
    if (OP == ISHMEM_OP_PROD) return acc * x;
    if (OP == ISHMEM_OP_MAX) return (x > acc) ? x : acc;
    if (OP == ISHMEM_OP_MIN) return (x < acc) ? x : acc;
    return acc;
}
/* bitwise operators only exist for integers */
template <typename T, int OP>
__device__ __forceinline__ T combine_bits(T acc, T x)
{
    if (OP == ISHMEM_OP_AND) return acc & x;
    if (OP == ISHMEM_OP_OR) return acc | x;
    return acc ^ x;
}
template <typename T, int OP, bool BITS = (OP >= ISHMEM_OP_AND)>
struct folder {
    static __device__ __forceinline__ T f(T a, T x) { return combine<T, OP>(a, x); }
};
template <typename T, int OP>
struct folder<T, OP, true> {
    static __device__ __forceinline__ T f(T a, T x) { return combine_bits<T, OP>(a, x); }
};
/* 8- and 16-bit integers are promoted to int by the arithmetic operators; sum and product are
 * taken in unsigned int (no signed overflow) and cut back to the element's width */
#define ISHMEMI_NARROW_FOLDER(T)                                                                   \
    template <int OP>                                                                              \
    struct folder<T, OP, false> {                                                                  \
        static __device__ __forceinline__ T f(T a, T x)                                            \
        {                                                                                          \
            if (OP == ISHMEM_OP_SUM) return (T)((unsigned)a + (unsigned)x);                        \
            if (OP == ISHMEM_OP_PROD) return (T)((unsigned)a * (unsigned)x);                       \
            return combine<T, OP>(a, x);                                                           \
        }                                                                                          \
    };                                                                                             \
    template <int OP>                                                                              \
    struct folder<T, OP, true> {                                                                   \
        static __device__ __forceinline__ T f(T a, T x)                                            \
        {                                                                                          \
            if (OP == ISHMEM_OP_AND) return (T)((unsigned)a & (unsigned)x);                        \
            if (OP == ISHMEM_OP_OR) return (T)((unsigned)a | (unsigned)x);                         \
            return (T)((unsigned)a ^ (unsigned)x);                                                 \
        }                                                                                          \
    };
ISHMEMI_NARROW_FOLDER(signed char)
ISHMEMI_NARROW_FOLDER(unsigned char)
ISHMEMI_NARROW_FOLDER(short)
ISHMEMI_NARROW_FOLDER(unsigned short)
#undef ISHMEMI_NARROW_FOLDER
/* signed integer sum/prod must wrap: do them unsigned */
template <int OP>
struct folder<int, OP, false> {
    static __device__ __forceinline__ int f(int a, int x)
    {
        if (OP == ISHMEM_OP_SUM) return (int)((unsigned)a + (unsigned)x);
        if (OP == ISHMEM_OP_PROD) return (int)((unsigned)a * (unsigned)x);
        return combine<int, OP>(a, x);
    }
};
template <int OP>
struct folder<long long, OP, false> {
    static __device__ __forceinline__ long long f(long long a, long long x)
    {
        if (OP == ISHMEM_OP_SUM) return (long long)((unsigned long long)a + (unsigned long long)x);
        if (OP == ISHMEM_OP_PROD) return (long long)((unsigned long long)a * (unsigned long long)x);
        return combine<long long, OP>(a, x);
    }
};

template <typename T>
union vec16 {
    uint4 v;
    T e[16 / sizeof(T)];
};

/* team index of a PE, or -1 */
__device__ __forceinline__ int team_index(const ishmemi_team &t, int pe)
{
    int d = pe - t.start;
    if (d < 0 || d % t.stride) return -1;
    d /= t.stride;
    return d < t.size ? d : -1;
}

/* Looks every team member up in the reachability table once and leaves, per team index,
 * the offset from the calling PE's heap to that member's heap in `delta` (shared memory,
 * ISHMEM_MAX_PES entries).  All threads call; ends with a block barrier.  Returns false
 * when a member is not reachable. */
__device__ __forceinline__ bool team_deltas(const ishmem_ctx_t *ctx, const ishmemi_team &t,
                                            long long *delta)
{
    __shared__ int bad;
    if (block_tid() == 0) bad = 0;
    __syncthreads();
    for (unsigned i = block_tid(); i < (unsigned)t.size; i += block_nthr()) {
        int pe = t.start + (int)i * t.stride;
        unsigned k = ((unsigned)pe < (unsigned)ctx->npes) ? ctx->reach[pe] : 0u;
        if (k == 0) bad = 1;
        else delta[i] = ctx->heap_delta[pe];
    }
    __syncthreads();
    const bool ok = (bad == 0);
    if (!ok && block_tid() == 0) latch_error(ctx, ISHMEM_ERR_INVALID_PE);
    return ok;
}

/* Vector body of a fold: 16-byte vectors [v0, v1) of the team's sources, combined in team
 * order, stored to ndst destinations.  VPT vectors per thread and iteration, B sources per
 * batch: VPT*B independent 16-byte loads are in flight before the first combine. */
template <typename T, int OP, int VPT, int B>
__device__ __forceinline__ void fold_vectors(const char *src, char *dest, const long long *delta, int tsize,
                                             int dst0, int ndst, size_t v0, size_t v1, unsigned tid,
                                             unsigned nthr)
{
    constexpr int EPV = 16 / sizeof(T);
    for (size_t v = v0 + tid; v < v1; v += (size_t)nthr * VPT) {
        vec16<T> acc[VPT];
#pragma unroll
        for (int u = 0; u < VPT; ++u)
            if (v + (size_t)u * nthr < v1) acc[u].v = ld16(src + delta[0] + (v + (size_t)u * nthr) * 16);
        for (int i = 1; i < tsize; i += B) {
            vec16<T> x[VPT][B];
#pragma unroll
            for (int u = 0; u < VPT; ++u)
#pragma unroll
                for (int k = 0; k < B; ++k)
                    if (i + k < tsize && v + (size_t)u * nthr < v1)
                        x[u][k].v = ld16(src + delta[i + k] + (v + (size_t)u * nthr) * 16);
#pragma unroll
            for (int u = 0; u < VPT; ++u)
#pragma unroll
                for (int k = 0; k < B; ++k)
                    if (i + k < tsize && v + (size_t)u * nthr < v1) {
#pragma unroll
                        for (int e = 0; e < EPV; ++e)
                            acc[u].e[e] = folder<T, OP>::f(acc[u].e[e], x[u][k].e[e]);
                    }
        }
        for (int q = 0; q < ndst; ++q) {
#pragma unroll
            for (int u = 0; u < VPT; ++u)
                if (v + (size_t)u * nthr < v1)
                    st16(dest + delta[dst0 + q] + (v + (size_t)u * nthr) * 16, acc[u].v);
        }
    }
}

/* Push `n` bytes at `src` to the `ndst` destinations dest + delta[q] (q = 0..ndst-1),
 * skipping q == skip: outer loop over addresses, inner loop over destinations, so that
 * consecutive stores go to different PEs (Section 3.7.2). */
__device__ __forceinline__ void push_bytes(char *dest, const long long *delta, int ndst, int skip,
                                           const char *src, size_t n, unsigned tid, unsigned nthr)
{
    const bool vec_ok = ((((uintptr_t)src | (uintptr_t)dest) & 15u) == 0);
    size_t nvec = vec_ok ? (n >> 4) : 0;
    size_t i = tid;
    for (; i + nthr < nvec; i += 2 * (size_t)nthr) {
        uint4 a = ld16(src + i * 16), b = ld16(src + (i + nthr) * 16);
        for (int q = 0; q < ndst; ++q) {
            if (q == skip) continue;
            st16(dest + delta[q] + i * 16, a);
            st16(dest + delta[q] + (i + nthr) * 16, b);
        }
    }
    for (; i < nvec; i += nthr) {
        uint4 a = ld16(src + i * 16);
        for (int q = 0; q < ndst; ++q)
            if (q != skip) st16(dest + delta[q] + i * 16, a);
    }
    for (size_t j = (nvec << 4) + tid; j < n; j += nthr) {
        unsigned char c = ldv<unsigned char>(src + j);
        for (int q = 0; q < ndst; ++q)
            if (q != skip) stv<unsigned char>(dest + delta[q] + j, c);
    }
}

/* Fold elements [begin, end) of the team's sources in team order and store the result in
 * the `ndst` destinations starting at team index dst0 (ndst = 1, dst0 = my index: the
 * duplicated algorithm; ndst = team size, dst0 = 0: the owner pushes to everybody).  src and
 * dest are the calling PE's local addresses; member i's copy is delta[i] bytes further.
 * 16-byte vectors when both buffers are 16-byte aligned, else element by element. */
template <typename T, int OP, int VPT = 1, int B = 4>
__device__ __forceinline__ void fold_range(const char *src, char *dest, const long long *delta,
                                           int tsize, int dst0, int ndst, size_t begin, size_t end,
                                           unsigned tid, unsigned nthr)
{
    constexpr int EPV = 16 / sizeof(T);
    const bool vec_ok = ((((uintptr_t)src | (uintptr_t)dest) & 15u) == 0);
    size_t vbeg = begin, vend = begin;
    if (vec_ok) {
        vbeg = (begin + EPV - 1) / EPV * EPV;
        vend = end / EPV * EPV;
        if (vbeg > vend) vbeg = vend = begin;
    }
    /* scalar edges: [begin, vbeg) and [vend, end) */
    for (size_t j = begin + tid; j < end; j += nthr) {
        if (j >= vbeg && j < vend) continue;
        T acc = ldv<T>(src + delta[0] + j * sizeof(T));
        for (int i = 1; i < tsize; ++i)
            acc = folder<T, OP>::f(acc, ldv<T>(src + delta[i] + j * sizeof(T)));
        for (int q = 0; q < ndst; ++q) stv<T>(dest + delta[dst0 + q] + j * sizeof(T), acc);
    }
    fold_vectors<T, OP, VPT, B>(src, dest, delta, tsize, dst0, ndst, vbeg / EPV, vend / EPV, tid, nthr);
}

/* Reduce through shared memory with TMA on both sides, called by every thread of the block:
 * for each chunk one elected thread bulk-loads the chunk of all `tsize` sources into one
 * stage (completing on one mbarrier), all threads fold the stage in team order into its
 * first tile, and the elected thread bulk-stores that tile to the `ndst` destinations
 * dest + delta[dst0 + q].  `nbytes` is a multiple of 16, src/dest 16-byte aligned, the ring
 * has 3 stages of tsize tiles.  The block handles chunks first, first+stride, ... of the range.
 * Returns 0, ISHMEM_ERR_TIMEOUT, or 1 when the staging is too small for this team (nothing
 * done). */
template <typename T, int OP>
__device__ __forceinline__ int bulk_fold_ring(const ishmem_ctx_t *ctx, const char *src, char *dest,
                                              const long long *delta, int tsize, int dst0, int ndst,
                                              size_t nbytes, ishmemx_staging_t st, size_t first = 0,
                                              size_t stride = 1)
{
    constexpr int EPV = 16 / sizeof(T);
    constexpr unsigned NST = 3;
    const unsigned tid = block_tid(), nthr = block_nthr();
    if (st.smem == nullptr || st.bytes < 128u + NST * 1024u * (unsigned)tsize) return 1;
    unsigned C = ((st.bytes - 128u) / (NST * (unsigned)tsize)) & ~1023u;
    if (C > 16384u) C = 16384u;
    const unsigned stage_bytes = C * (unsigned)tsize;
    /* this block takes chunks first, first + stride, ... of the range (round-robin with the
     * other blocks of the launch) */
    const size_t total = (nbytes + C - 1) / C;
    const size_t nchunks = total > first ? (total - first + stride - 1) / stride : 0;
    char *stage0 = (char *)st.smem + 128;
    const unsigned bar0 = smem_u32(st.smem), sm0 = smem_u32(stage0);
    __shared__ int fail;
    if (tid == 0) {
        fail = 0;
        for (unsigned k = 0; k < NST; ++k) mbar_init(bar0 + 8 * k, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    __syncthreads();
    auto chunk_off = [&](size_t c) -> size_t { return (first + c * stride) * C; };
    auto chunk_bytes = [&](size_t c) -> unsigned {
        size_t left = nbytes - chunk_off(c);
        return left < C ? (unsigned)left : C;
    };
    auto issue_load = [&](size_t c) {
        const unsigned sidx = (unsigned)(c % NST), b = chunk_bytes(c);
        mbar_expect_tx(bar0 + 8 * sidx, b * (unsigned)tsize);
        for (int i = 0; i < tsize; ++i)
            bulk_g2s(sm0 + sidx * stage_bytes + (unsigned)i * C, src + delta[i] + chunk_off(c), b,
                     bar0 + 8 * sidx);
    };
    size_t issued = 0;
    if (tid == 0)
        for (; issued < nchunks && issued + 1 < NST; ++issued) issue_load(issued);
    size_t c = 0;
    for (; c < nchunks; ++c) {
        const unsigned sidx = (unsigned)(c % NST);
        const bool ok = mbar_wait(bar0 + 8 * sidx, (unsigned)((c / NST) & 1), ctx->wait_limit_ns);
        if (!ok) fail = 1;
        const unsigned b = chunk_bytes(c);
        char *tile = stage0 + (size_t)sidx * stage_bytes;
        if (ok)
            for (unsigned v = tid; v < (b >> 4); v += nthr) {
                vec16<T> acc;
                acc.v = *(const uint4 *)(tile + (size_t)v * 16);
                for (int i = 1; i < tsize; ++i) {
                    vec16<T> x;
                    x.v = *(const uint4 *)(tile + (size_t)i * C + (size_t)v * 16);
#pragma unroll
                    for (int e = 0; e < EPV; ++e) acc.e[e] = folder<T, OP>::f(acc.e[e], x.e[e]);
                }
                *(uint4 *)(tile + (size_t)v * 16) = acc.v;
            }
        fence_proxy_async(); /* the folded tile is read by the bulk stores below */
        __syncthreads();
        if (fail) break;
        if (tid == 0) {
            for (int q = 0; q < ndst; ++q)
                bulk_s2g(dest + delta[dst0 + q] + chunk_off(c), sm0 + sidx * stage_bytes, b);
            bulk_commit();
            if (issued < nchunks) {
                bulk_wait_read<1>(); /* the stores of chunk c-1 have read their stage: refill it */
                issue_load(issued);
                ++issued;
            }
        }
    }
    if (tid == 0) {
        if (fail) {
            latch_error(ctx, ISHMEM_ERR_TIMEOUT);
            for (size_t k = c; k < issued; ++k)
                mbar_wait(bar0 + 8 * (unsigned)(k % NST), (unsigned)((k / NST) & 1), ctx->wait_limit_ns);
        }
        bulk_wait<0>();
        fence_proxy_async();
        for (unsigned k = 0; k < NST; ++k) mbar_inval(bar0 + 8 * k);
    }
    __syncthreads();
    return fail ? ISHMEM_ERR_TIMEOUT : 0;
}

/* work-group push of n bytes to ndst destinations dest + delta[q] (q != skip); delta lives in
 * shared memory.  TMA ring for the aligned body when staging is given, else loads/stores with
 * the destinations in the inner loop (see push_bytes).  With stride > 1 the caller is block
 * `first` of `stride` blocks that share the range chunk by chunk. */
__device__ __forceinline__ int wg_push(const ishmem_ctx_t *ctx, char *dest, const long long *delta, int ndst,
                                       int skip, const char *src, size_t n, ishmemx_staging_t st,
                                       size_t first = 0, size_t stride = 1, size_t tile = 16384)
{
    const unsigned tid = threadIdx.x + blockDim.x * (threadIdx.y + blockDim.y * threadIdx.z);
    const unsigned nthr = blockDim.x * blockDim.y * blockDim.z;
    const bool congruent = ((((uintptr_t)dest - (uintptr_t)src) & 15u) == 0);
    if (st.smem != nullptr && st.bytes >= 128u + 2048u && congruent && n >= ISHMEMI_BULK_MIN_BYTES) {
        size_t head = (size_t)((16u - ((unsigned)(uintptr_t)dest & 15u)) & 15u);
        size_t body = (n - head) & ~(size_t)15;
        size_t tail = n - head - body;
        if (first == 0) {
            push_bytes(dest, delta, ndst, skip, src, head, tid, nthr);
            push_bytes(dest + head + body, delta, ndst, skip, src + head + body, tail, tid, nthr);
        }
        fence_proxy_async();
        __syncthreads();
        __shared__ int rc_sh;
        if (tid == 0)
            rc_sh = bulk_copy_ring(ctx, dest + head, src + head, body, st, true, delta, ndst, skip, first, stride);
        __syncthreads();
        return rc_sh;
    }
    /* loads/stores: tiles of `tile` bytes (a multiple of 16) dealt round-robin (the whole range
     * when stride is 1) */
    if (stride == 1) {
        push_bytes(dest, delta, ndst, skip, src, n, tid, nthr);
    } else {
        for (size_t o = first * tile; o < n; o += stride * tile)
            push_bytes(dest + o, delta, ndst, skip, src + o, (n - o < tile) ? n - o : tile, tid, nthr);
    }
    return 0;
}

} /* namespace ishmemi */

/* The collectives below are called by ONE work-group per team member, every member
 * calling with the same arguments (dest/src: local addresses of symmetric objects). */

/* broadcast: the root pushes its source into every member's dest, then the team
 * synchronises, so that on return dest is complete on the calling PE.  `root` is a team
 * index. */
__device__ __forceinline__ int ishmemx_broadcastmem_work_group(const ishmem_ctx_t *ctx,
                                                               ishmem_team_t team, void *dest,
                                                               const void *src, size_t nbytes,
                                                               int root)
{
    __shared__ long long delta[ISHMEM_MAX_PES];
    const ishmemi_team t = ctx->teams[team];
    const int me = ishmemi::team_index(t, ctx->my_pe);
    const bool ok = ishmemi::team_deltas(ctx, t, delta);
    if (ok && me == root)
        ishmemi::push_bytes((char *)dest, delta, t.size, ctx->bcast_root_dest ? -1 : root,
                            (const char *)src, nbytes, ishmemi::block_tid(), ishmemi::block_nthr());
    int rc = ishmemx_team_sync_work_group(ctx, team);
    return ok ? rc : ISHMEM_ERR_INVALID_PE;
}

/* fcollect: every member pushes its source into block `my index` of every member's dest,
 * then the team synchronises. */
__device__ __forceinline__ int ishmemx_fcollectmem_work_group(const ishmem_ctx_t *ctx,
                                                              ishmem_team_t team, void *dest,
                                                              const void *src, size_t nbytes)
{
    __shared__ long long delta[ISHMEM_MAX_PES];
    const ishmemi_team t = ctx->teams[team];
    const int me = ishmemi::team_index(t, ctx->my_pe);
    const bool ok = ishmemi::team_deltas(ctx, t, delta);
    if (ok && me >= 0)
        ishmemi::push_bytes((char *)dest + (size_t)me * nbytes, delta, t.size, -1, (const char *)src,
                            nbytes, ishmemi::block_tid(), ishmemi::block_nthr());
    int rc = ishmemx_team_sync_work_group(ctx, team);
    return ok ? rc : ISHMEM_ERR_INVALID_PE;
}

/* collect: every member contributes `my_nbytes` bytes (they may differ); every member's dest ends
 * up with the concatenation in team order.  The sizes are exchanged first -- each member stores
 * its size into a slot of every member's internal region and the team synchronises -- then every
 * member pushes its source to its offset in every dest, and a second synchronisation completes
 * the call.  *total (may be nullptr) receives the gathered size. */
__device__ __forceinline__ int ishmemx_collectmem_work_group(const ishmem_ctx_t *ctx, ishmem_team_t team, void *dest,
                                                             const void *src, size_t my_nbytes, size_t *total = nullptr)
{
    __shared__ long long delta[ISHMEM_MAX_PES];
    __shared__ unsigned long long my_offset, all_bytes;
    const ishmemi_team t = ctx->teams[team];
    const int me = ishmemi::team_index(t, ctx->my_pe);
    const bool ok = ishmemi::team_deltas(ctx, t, delta) && me >= 0;
    const unsigned tid = ishmemi::block_tid(), nthr = ishmemi::block_nthr();
    if (ok)
        for (unsigned i = tid; i < (unsigned)t.size; i += nthr) {
            const int pe = t.start + (int)i * t.stride;
            unsigned long long *slot = (unsigned long long *)((char *)(ctx->collect_sizes + me) +
                                                              (long long)(pe - ctx->my_pe) * ctx->internal_stride);
            ishmemi::st_relaxed(slot, (unsigned long long)my_nbytes);
        }
    int rc = ishmemx_team_sync_work_group(ctx, team); /* release/acquire: all sizes have arrived */
    if (ok && rc == 0) {
        if (tid == 0) {
            unsigned long long off = 0, sum = 0;
            for (int i = 0; i < t.size; ++i) {
                const unsigned long long n = ishmemi::ld_relaxed(ctx->collect_sizes + i);
                if (i < me) off += n;
                sum += n;
            }
            my_offset = off;
            all_bytes = sum;
        }
        __syncthreads();
        ishmemi::push_bytes((char *)dest + my_offset, delta, t.size, -1, (const char *)src, my_nbytes, tid, nthr);
        if (total) *total = (size_t)all_bytes;
    }
    int rc2 = ishmemx_team_sync_work_group(ctx, team);
    return !ok ? ISHMEM_ERR_INVALID_PE : (rc ? rc : rc2);
}

/* alltoall: every member stores block q of its source into block `my index` of member q's dest
 * (push, destinations in the inner loop like broadcast), then the team synchronises. */
__device__ __forceinline__ int ishmemx_alltoallmem_work_group(const ishmem_ctx_t *ctx, ishmem_team_t team,
                                                              void *dest, const void *src, size_t nbytes)
{
    __shared__ long long delta[ISHMEM_MAX_PES];
    const ishmemi_team t = ctx->teams[team];
    const int me = ishmemi::team_index(t, ctx->my_pe);
    const bool ok = ishmemi::team_deltas(ctx, t, delta);
    if (ok && me >= 0)
        for (int q = 0; q < t.size; ++q)
            ishmemi::copy_bytes((char *)dest + delta[q] + (size_t)me * nbytes, (const char *)src + (size_t)q * nbytes,
                                nbytes, ishmemi::block_tid(), ishmemi::block_nthr());
    int rc = ishmemx_team_sync_work_group(ctx, team);
    return ok ? rc : ISHMEM_ERR_INVALID_PE;
}

/* reduce (the paper's small-message algorithm): after an entry sync (all sources ready)
 * every PE folds all sources itself -- address range split across its threads, vector
 * loads of the local and the remote sources, vector store to its own dest; an exit sync
 * lets sources be reused.  Folded in team order. */
template <typename T, int OP>
__device__ __forceinline__ int ishmemx_reduce_work_group(const ishmem_ctx_t *ctx, ishmem_team_t team,
                                                         T *dest, const T *src, size_t nreduce)
{
    __shared__ long long delta[ISHMEM_MAX_PES];
    const ishmemi_team t = ctx->teams[team];
    const int me = ishmemi::team_index(t, ctx->my_pe);
    const bool ok = ishmemi::team_deltas(ctx, t, delta);
    int rc = ishmemx_team_sync_work_group(ctx, team);
    if (ok && rc == 0 && me >= 0)
        ishmemi::fold_range<T, OP>((const char *)src, (char *)dest, delta, t.size, me, 1, 0, nreduce,
                                   ishmemi::block_tid(), ishmemi::block_nthr());
    int rc2 = ishmemx_team_sync_work_group(ctx, team);
    return !ok ? ISHMEM_ERR_INVALID_PE : (rc ? rc : rc2);
}

#endif /* ISHMEM_DEVICE_CUH */
