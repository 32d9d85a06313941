/*
 * ishmem.h -- C ABI of libishmem.so: GPU-initiated OpenSHMEM-style communication on a
 * symmetric heap, after Intel SHMEM (arXiv 2409.20476), for one NVIDIA B200 (sm_100a).
 *
 * Execution model.  One process hosts `npes` logical processing elements (PEs).  Each
 * PE owns one slice of `heap_bytes` of a single device allocation: its symmetric heap
 * (Section 2.3: PEs 0..npes-1, identical layout on every PE, different contents;
 * Section 3.5: the heap lives in GPU memory).  Because every PE lives in this process,
 * host calls that OpenSHMEM makes "as a PE" carry the calling PE as their first
 * argument `my_pe`; collectives are called once for the whole team.
 *
 * Addresses.  A *symmetric address* is the device address of the object in PE 0's
 * slice, as returned by ishmem_malloc; the library translates it to the addressed PE
 * with `addr - heap_base[0] + heap_base[pe]` (Section 3.7.1, the ishmem_long_p
 * walk-through).  Unless stated otherwise: the `dest` of a put, the `src` of a get,
 * atomic targets, signal words and all collective buffers must be symmetric; the
 * other side may be a symmetric address (meaning my_pe's copy) or any other device
 * pointer.  All data pointers are DEVICE pointers unless the parameter is documented
 * as host memory.  The library never takes ownership of caller memory; memory from
 * ishmem_malloc belongs to the library until ishmem_free / ishmem_finalize.
 *
 * Ordering.  Host-initiated operations of PE p are enqueued on PE p's CUDA stream and
 * return at once (stream-ordered); team collectives and SPMD launches run on the
 * team stream, after everything already enqueued on the member PEs' streams.
 * ishmem_quiet / ishmem_barrier_all are the completion points (Section 3.7.2: barrier
 * = quiet + sync).  Overlapping src/dest ranges on one PE are undefined.
 *
 * Errors.  Functions returning int give ISHMEM_OK (0) or a negative ishmem_status;
 * nothing is enqueued when an argument check fails.  Pointer-returning functions
 * give NULL on failure.  Device-side waits are bounded: when a wait gives up it
 * latches ISHMEM_ERR_TIMEOUT in a device status word that ishmemx_status() reads.
 * There is no CPU fallback anywhere: without a CUDA device ishmem_init fails.
 */
#ifndef ISHMEM_H
#define ISHMEM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ISHMEM_MAX_PES 64

typedef enum ishmem_status {
    ISHMEM_OK = 0,
    ISHMEM_ERR_INVALID_PE = -1,     /* PE outside 0..npes-1, or outside the team */
    ISHMEM_ERR_NOT_SYMMETRIC = -2,  /* address range is not inside the symmetric heap */
    ISHMEM_ERR_ALIGN = -3,          /* address not aligned for the element type */
    ISHMEM_ERR_OOM = -4,            /* symmetric heap or device memory exhausted */
    ISHMEM_ERR_TIMEOUT = -5,        /* a bounded device-side wait gave up */
    ISHMEM_ERR_NOT_CORESIDENT = -6, /* a launch whose blocks wait on one another does not fit */
    ISHMEM_ERR_CUDA = -7,           /* a CUDA runtime call failed (see ishmemx_last_cuda_error) */
    ISHMEM_ERR_ARG = -8,            /* other invalid argument */
    ISHMEM_ERR_NOT_INITIALIZED = -9
} ishmem_status;

/* Teams (Section 3.7.2 uses ISHMEM_TEAM_SHARED; OpenSHMEM 1.5 teams API).  A team is the
 * PE set {start + i*stride}.  WORLD and SHARED both name all PEs here: every PE is
 * reachable by load/store from every other. */
typedef int ishmem_team_t;
#define ISHMEM_TEAM_WORLD 0
#define ISHMEM_TEAM_SHARED 1
#define ISHMEM_TEAM_INVALID (-1)
#define ISHMEM_MAX_TEAMS 16

/* signal operators of put_signal, comparisons of wait_until */
#define ISHMEM_SIGNAL_SET 0
#define ISHMEM_SIGNAL_ADD 1
#define ISHMEM_CMP_EQ 0
#define ISHMEM_CMP_NE 1
#define ISHMEM_CMP_GT 2
#define ISHMEM_CMP_GE 3
#define ISHMEM_CMP_LT 4
#define ISHMEM_CMP_LE 5

/* thread-collaboration level of the device-side copy routines (Section 3.6: work-item =
 * one thread, sub-group = one warp of 32 lanes, work-group = one thread block). */
#define ISHMEMX_WORK_ITEM 0
#define ISHMEMX_SUB_GROUP 1
#define ISHMEMX_WORK_GROUP 2       /* 16-byte vector loads/stores by all threads */
#define ISHMEMX_WORK_GROUP_BULK 3  /* work-group; large aligned blocks go through TMA bulk copies */
#define ISHMEMX_WORK_GROUP_ENGINE 4 /* work-group; the leader asks the host proxy to start the copy engine */

/* reduction operators and element types of the generic reduce entry point */
#define ISHMEM_OP_SUM 0
#define ISHMEM_OP_MAX 1
#define ISHMEM_OP_MIN 2
#define ISHMEM_OP_PROD 3
#define ISHMEM_OP_AND 4
#define ISHMEM_OP_OR 5
#define ISHMEM_OP_XOR 6
#define ISHMEM_T_INT32 0
#define ISHMEM_T_INT64 1
#define ISHMEM_T_FLOAT 2
#define ISHMEM_T_DOUBLE 3
#define ISHMEM_T_UINT32 4
#define ISHMEM_T_UINT64 5
#define ISHMEM_T_INT8 6
#define ISHMEM_T_UINT8 7
#define ISHMEM_T_INT16 8
#define ISHMEM_T_UINT16 9

/* reduce algorithms (Section 3.7.2, "Reduction") */
#define ISHMEMX_REDUCE_AUTO 0
#define ISHMEMX_REDUCE_DUPLICATED 1 /* every PE folds all sources itself, no inter-PE sync */
#define ISHMEMX_REDUCE_SPLIT 2      /* addresses split across PEs; the owner folds and pushes */

/* ------------------------------------------------------------------ lifecycle --- */

/* Host-only (Section 3.6).  Creates `npes` PEs (1..ISHMEM_MAX_PES) on the current CUDA
 * device, each with `heap_bytes` of symmetric heap (rounded up to 256 B), zero-filled.
 * ishmem_init allocates the heap with cudaMalloc; ishmemx_init_external uses
 * npes*heap_bytes bytes at `base` (device memory, 256-byte aligned, owned by the caller,
 * e.g. a torch tensor; cf. the external-heap registration of Section 3.5) and does
 * not clear it.  ISHMEM_ERR_ARG if already initialised.  ishmem_init(npes, 0) takes the heap
 * size per PE from the environment variable ISHMEM_SYMMETRIC_SIZE (bytes).  Other variables read
 * at initialisation: ISHMEM_CUTOVER_{PUT,PUT_UPTO,BCAST,FCOLLECT,WORK_GROUP} (bytes, "never" or "always";
 * see ishmemx_set_cutover), ISHMEM_WAIT_TIMEOUT_NS (see ishmemx_set_wait_limit_ns) and the
 * initial values of the launch-shape switches (ISHMEM_JACOBI_SPLIT, _JACOBI_FUSE, _JACOBI_WIDE,
 * ISHMEM_REDUCE_BULK, ISHMEM_BULK_SMEM, ISHMEM_PUSH_SHAPE; see ishmemx_set_option).  No variable is read later. */
int ishmem_init(int npes, size_t heap_bytes);
int ishmemx_init_external(int npes, size_t heap_bytes, void *base);
/* Waits for all streams, frees everything the library allocated. */
int ishmem_finalize(void);
int ishmem_n_pes(void);                /* 0 when not initialised */
size_t ishmemx_heap_bytes(void);
/* Launch-shape switches.  Each has a default that the library picks from measurement; a test or
 * a size sweep selects another form through ishmemx_set_option, never through the process
 * environment at call time.  The environment variable named beside an option is read ONCE, by
 * ishmem_init / ishmemx_init_external, and only sets the option's initial value; a later
 * ishmemx_set_option wins.  All options are reset by the next initialisation.
 *   ISHMEMX_OPT_JACOBI_SPLIT (ISHMEM_JACOBI_SPLIT=rows|columns): 0 = the library's choice (for
 *       threads = 0 and an even nx: launch-ordered sweeps; else the persistent kernel, strips cut
 *       by rows), 1 = persistent kernel with the strips cut by rows, 2 = by ranges of column
 *       tiles.
 *   ISHMEMX_OPT_JACOBI_FUSE (ISHMEM_JACOBI_FUSE=0..6): sweeps per launch of the launch-ordered
 *       form: 1 = the library's choice, up to six (default), 0 = always one, 2 .. 6 = at most
 *       that many.
 *   ISHMEMX_OPT_JACOBI_WIDE (ISHMEM_JACOBI_WIDE=0|1): columns per lane in the multi-sweep launches:
 *       -1 = four where nx is a multiple of 4 and the grid gives every SM its blocks (default),
 *       0 = two, 1 = four (nx a multiple of 4, else two).
 *   ISHMEMX_OPT_REDUCE_BULK (ISHMEM_REDUCE_BULK=0|1): 1 = large split reductions go through the
 *       shared-memory TMA fold ring instead of one tile per block (default 0).
 *   ISHMEMX_OPT_BULK_SMEM (ISHMEM_BULK_SMEM=bytes): shared-memory staging per block of the
 *       ISHMEMX_WORK_GROUP_BULK level (default 192 KiB + 128, capped by the device limit).
 *   ISHMEMX_OPT_PUSH_SHAPE (ISHMEM_PUSH_SHAPE=0|1|2): launch shape of host-called broadcast and
 *       fcollect by stores: 1 = fan-out tiles (a thread stores each vector it loads to every
 *       destination), 2 = one block per (tile, source member, destination), each a plain copy,
 *       0 = by measurement (default: the second for messages of at least 4 MiB on teams of up to
 *       6 members, where it is up to 25 % faster; the first otherwise).
 * ishmemx_set_option returns ISHMEM_ERR_ARG for an unknown option or a value outside its range;
 * ishmemx_get_option returns the current value (0 for an unknown option). */
#define ISHMEMX_OPT_JACOBI_SPLIT 0
#define ISHMEMX_OPT_JACOBI_FUSE 1
#define ISHMEMX_OPT_JACOBI_WIDE 2
#define ISHMEMX_OPT_REDUCE_BULK 3
#define ISHMEMX_OPT_BULK_SMEM 4
#define ISHMEMX_OPT_PUSH_SHAPE 5
#define ISHMEMX_OPT_COUNT 6
int ishmemx_set_option(int option, long long value);
long long ishmemx_get_option(int option);
/* Device pointer to PE `pe`'s context (ishmem_ctx_t, see ishmem_device.cuh), to hand to
 * user kernels; the array of all contexts starts at ishmemx_ctx(0).  NULL on error. */
void *ishmemx_ctx(int pe);
/* Replace PE `pe`'s stream (pe = -1: the team stream) by a caller-owned cudaStream_t. */
int ishmemx_set_stream(int pe, void *cuda_stream);
void *ishmemx_get_stream(int pe);
const char *ishmem_strerror(int status);
const char *ishmemx_last_cuda_error(void);
/* Reads (and with clear != 0 resets) the device status word latched by bounded waits.
 * Blocks until all library streams are idle. */
int ishmemx_status(int clear);
/* Number of kernels the library has launched since ishmem_init. */
unsigned long long ishmemx_launch_count(void);
/* Time bound, in nanoseconds, of every device-side wait (default 2e9 = two seconds). */
int ishmemx_set_wait_limit_ns(uint64_t ns);

/* --------------------------------------------------- symmetric memory (host only) --- */

/* Collective allocation: the same offset on every PE (Section 2.3).  256-byte aligned
 * (ishmem_align: `alignment` a power of two).  Returns the symmetric address (PE 0's
 * copy) or NULL when the heap is exhausted.  ishmem_calloc zero-fills every PE's copy.
 * ishmem_free(NULL) is a no-op; freeing a pointer not returned by these is an error. */
void *ishmem_malloc(size_t size);
void *ishmem_calloc(size_t count, size_t size);
void *ishmem_align(size_t alignment, size_t size);
int ishmem_free(void *ptr);
/* PE `pe`'s copy of the symmetric object (device pointer usable by loads and stores from
 * any kernel: Section 3.3, every peer heap is mapped).  NULL if not symmetric. */
void *ishmem_ptr(const void *sym, int pe);
/* Staging helpers (host <-> one PE's copy), enqueued on that PE's stream.  `host` is HOST
 * memory; pinned memory makes the copy asynchronous. */
int ishmemx_heap_write(int pe, void *sym_dest, const void *host, size_t nbytes);
int ishmemx_heap_read(int pe, void *host, const void *sym_src, size_t nbytes);

/* ----------------------------------------------------------- RMA (Section 3.7.1) --- */

/* Host-initiated put/get of `nbytes`: PE my_pe copies src -> dest@pe (put) or src@pe ->
 * dest (get).  Subject to the cutover (Sections 3.2, 4): below the tuned size a kernel of
 * cooperating threads does loads/stores, above it the copy engine (cudaMemcpyAsync on a
 * side stream) is started.  The blocking forms order later work of my_pe's stream after
 * the transfer; the _nbi forms only guarantee completion after ishmem_quiet(my_pe). */
int ishmem_putmem(int my_pe, void *dest, const void *src, size_t nbytes, int pe);
int ishmem_getmem(int my_pe, void *dest, const void *src, size_t nbytes, int pe);
int ishmem_putmem_nbi(int my_pe, void *dest, const void *src, size_t nbytes, int pe);
int ishmem_getmem_nbi(int my_pe, void *dest, const void *src, size_t nbytes, int pe);

/* Typed forms: `nelems` elements; addresses must be aligned to the element size. */
#define ISHMEM_DECL_RMA(NAME, T)                                                              \
    int ishmem_##NAME##_put(int my_pe, T *dest, const T *src, size_t nelems, int pe);         \
    int ishmem_##NAME##_get(int my_pe, T *dest, const T *src, size_t nelems, int pe);         \
    int ishmem_##NAME##_put_nbi(int my_pe, T *dest, const T *src, size_t nelems, int pe);     \
    int ishmem_##NAME##_get_nbi(int my_pe, T *dest, const T *src, size_t nelems, int pe);     \
    /* scalar store / load of one element at a symmetric address (the ishmem_long_p example \
     * of Section 3.7.1).  g blocks the host and writes the value to HOST memory. */         \
    int ishmem_##NAME##_p(int my_pe, T *dest, T value, int pe);                               \
    int ishmem_##NAME##_g(int my_pe, T *value_out_host, const T *src, int pe);
ISHMEM_DECL_RMA(float, float)
ISHMEM_DECL_RMA(double, double)
ISHMEM_DECL_RMA(int, int)
ISHMEM_DECL_RMA(long, long)
ISHMEM_DECL_RMA(int32, int32_t)
ISHMEM_DECL_RMA(int64, int64_t)
ISHMEM_DECL_RMA(uint8, uint8_t)
ISHMEM_DECL_RMA(uint32, uint32_t)
ISHMEM_DECL_RMA(uint64, uint64_t)
#undef ISHMEM_DECL_RMA

/* Strided put / get (OpenSHMEM iput / iget; the strided form that Section 3.7.1 lists): element k of
 * the source, taken every `sst` elements, becomes element k*dst of the destination, k = 0 ..
 * nelems-1.  Strides are in elements and at least 1; elem_size is 1, 2, 4, 8 or 16 bytes and both
 * addresses must be aligned to it.  Symmetric side and ordering as for ishmem_putmem /
 * ishmem_getmem; always a kernel of cooperating threads (no cutover). */
int ishmemx_iputmem(int my_pe, void *dest, const void *src, size_t dst, size_t sst, size_t nelems,
                    size_t elem_size, int pe);
int ishmemx_igetmem(int my_pe, void *dest, const void *src, size_t dst, size_t sst, size_t nelems,
                    size_t elem_size, int pe);
#define ISHMEM_DECL_STRIDED(NAME, T)                                                          \
    int ishmem_##NAME##_iput(int my_pe, T *dest, const T *src, size_t dst, size_t sst,        \
                             size_t nelems, int pe);                                          \
    int ishmem_##NAME##_iget(int my_pe, T *dest, const T *src, size_t dst, size_t sst,        \
                             size_t nelems, int pe);
ISHMEM_DECL_STRIDED(float, float)
ISHMEM_DECL_STRIDED(double, double)
ISHMEM_DECL_STRIDED(int, int)
ISHMEM_DECL_STRIDED(long, long)
ISHMEM_DECL_STRIDED(int32, int32_t)
ISHMEM_DECL_STRIDED(int64, int64_t)
ISHMEM_DECL_STRIDED(uint8, uint8_t)
ISHMEM_DECL_STRIDED(uint32, uint32_t)
ISHMEM_DECL_STRIDED(uint64, uint64_t)
#undef ISHMEM_DECL_STRIDED

/* Explicit thread-collaborative variants (Section 3.6; experiments of Section 4): a
 * kernel of `groups` blocks x `threads` threads is launched on my_pe's stream; the message
 * is cut into one contiguous slice per collaboration unit (thread / warp / block,
 * `level` = ISHMEMX_WORK_ITEM..ISHMEMX_WORK_GROUP_ENGINE) and every unit calls the device
 * routine ishmem_putmem / ishmemx_putmem_sub_group / ishmemx_putmem_work_group /
 * ishmemx_putmem_engine_work_group once on its slice.  threads in 1..1024, groups >= 1.
 * ISHMEMX_WORK_GROUP_ENGINE needs a running proxy (ISHMEM_ERR_ARG otherwise) and blocks the host
 * until the kernel has finished: nothing may be queued behind a kernel that waits for the proxy
 * (see ishmemx_proxy_start). */
int ishmemx_putmem_on_device(int my_pe, void *dest, const void *src, size_t nbytes, int pe,
                             int level, int threads, int groups);
int ishmemx_getmem_on_device(int my_pe, void *dest, const void *src, size_t nbytes, int pe,
                             int level, int threads, int groups);
/* The copy-engine path alone (cudaMemcpyAsync on the side stream, joined back into
 * my_pe's stream). */
int ishmemx_putmem_copy_engine(int my_pe, void *dest, const void *src, size_t nbytes, int pe);
int ishmemx_getmem_copy_engine(int my_pe, void *dest, const void *src, size_t nbytes, int pe);
/* SPMD form: ONE launch on the team stream in which every PE p runs the same device call
 * with target (p + shift) mod npes -- shift 1 is the ring pattern, shifts 1..npes-1 in turn
 * the all-pairs pattern.  `groups` blocks per PE; groups == 0 lets the library size the grid so
 * that every block gets one tile of threads x 128 bytes (blocks start in index order and sweep one
 * short window of memory together: the fastest shape for large messages on B200, and what
 * ishmem_putmem chooses by itself).  dest and src are symmetric. */
int ishmemx_putmem_spmd(void *dest, const void *src, size_t nbytes, int shift, int level,
                        int threads, int groups);
int ishmemx_getmem_spmd(void *dest, const void *src, size_t nbytes, int shift, int level,
                        int threads, int groups);
/* Same pattern through the copy engine: npes cudaMemcpyAsync calls on the side stream. */
int ishmemx_putmem_spmd_copy_engine(void *dest, const void *src, size_t nbytes, int shift);

/* Cutover sizes in bytes (Section 4: tuned from measurement; for the collaborative calls
 * it depends on the number of threads).  which: 0 = host-initiated put/get, 1 = broadcast,
 * 2 = fcollect, 3 = device-initiated work-group put/get (takes effect while the host proxy of
 * ishmemx_proxy_start runs).  SIZE_MAX = never use the copy engine, 0 = always.
 * which = 5 is the upper end of the host-initiated band: ishmem_putmem / getmem (and _nbi) use
 * the engine for cutover 0 <= nbytes < cutover 5 and the tiled kernel outside it (SIZE_MAX = no
 * upper end).  Defaults, from the size sweep on B200: the engine wins from 4 MiB to 32 MiB and
 * loses or ties from 64 MiB on, so which = 0 is 4 MiB and which = 5 is 64 MiB; SIZE_MAX for
 * 1, 2 and 3 (environment overrides: ISHMEM_CUTOVER_PUT, _PUT_UPTO, _BCAST, _FCOLLECT,
 * _WORK_GROUP).
 * which = 4 is not a threshold but the hybrid head: a blocking work-group put/get above cutover 3
 * gives the engine everything past the first `nbytes` bytes (rounded down to 256) and copies
 * that head itself meanwhile, hiding the engine's start-up; 0 (the default) = engine only. */
int ishmemx_set_cutover(int which, size_t nbytes);
size_t ishmemx_get_cutover(int which);
/* Picks the cutover from measurement on this device (Section 4 leaves it to tuning), for
 * which = 0 (host-initiated put, PE 0 -> PE 1, CUDA events) or which = 3 (device-initiated put
 * by ONE work-group of `threads` threads, timed inside the kernel; needs a running proxy).
 * Times both paths at 4 KiB, 16 KiB, ... (which = 0: 4 KiB, 8 KiB, ...) up to max_bytes (two
 * temporary symmetric buffers of max_bytes are allocated and freed: ISHMEM_ERR_OOM if the heap
 * has no room).  which = 3: sets the cutover to the smallest size from which the copy engine is at
 * least as fast at every larger size tried, or SIZE_MAX when it never is.  which = 0: gives the
 * engine the longest run of consecutive sizes at which it is at least as fast -- cutover 0 becomes
 * the first size of that run and cutover 5 the first size after it at which the kernel wins
 * (SIZE_MAX when the run reaches max_bytes; both SIZE_MAX when the engine never wins).  The
 * lower bound is also written to HOST *chosen (may be NULL).  Blocks the host. */
int ishmemx_tune_cutover(int which, int threads, size_t max_bytes, size_t *chosen);

/* ------------------------------------- reverse offload: GPU -> host requests (Section 3.4) --- */

/* Starts / stops the host proxy thread and its request ring.  While it runs, device code can
 * hand copies to the copy engine (ishmemx_putmem_engine_work_group and the cutover of
 * ishmemx_putmem_work_group, see ishmem_device.cuh): a GPU thread writes one 64-byte request
 * into a ring in pinned host memory (one fetch-and-increment to allocate the slot, stores
 * only), the proxy issues cudaMemcpyAsync on the issuing PE's copy-engine stream, and the reply
 * is written behind the copy in stream order into a word the GPU thread polls.  Both calls
 * block until the device is idle; ishmem_finalize stops a running proxy.  Allocates pinned host
 * memory (ring of 8192 requests, 65536 reply words).
 * Progress: a kernel that waits for the proxy depends on the proxy's streams being served while
 * it runs.  CUDA multiplexes streams onto a few hardware queues (8 by default); work already
 * queued BEHIND the waiting kernel, on a stream that shares a queue with a proxy stream, blocks
 * the proxy's copy, and the wait then ends only by its time limit (ISHMEM_ERR_TIMEOUT latched,
 * nothing hangs).  Either queue nothing behind such a kernel, or start the process with
 * CUDA_DEVICE_MAX_CONNECTIONS=32 (read when the CUDA context is created; measured on B200:
 * 32 launches queued back to back, no time-outs with 32 queues, sporadic ones with 8).
 * ishmemx_proxy_start reads one environment variable, once: ISHMEM_PROXY_NO_STREAM_MEMOPS (set to
 * anything) makes the replies 8-byte copies even where stream memory operations exist. */
int ishmemx_proxy_start(void);
int ishmemx_proxy_stop(void);
/* Requests served and copies started since ishmemx_proxy_start (HOST pointers, may be NULL);
 * *uses_stream_memops = 1 when replies are written by stream memory operations, 0 when by
 * 8-byte copies.  ISHMEM_ERR_ARG when no proxy runs. */
int ishmemx_proxy_stats(uint64_t *requests_served, uint64_t *copies_started, int *uses_stream_memops);
/* Ring measurement: `blocks` x `threads` GPU threads each post `iters` no-op requests.
 * mode 0: each request waits for its reply -> *mean_rtt_ns = mean GPU -> host -> GPU round trip
 * (device global timer).  mode 1: no replies except for each thread's last request ->
 * *requests_per_second = requests / time as seen from the GPU (HOST pointers, may be NULL).
 * Needs a running proxy.  Blocks the host. */
int ishmemx_ring_benchmark(int mode, int blocks, int threads, int iters, double *mean_rtt_ns,
                           double *requests_per_second);

/* ------------------------------------------- signalling, ordering, synchronisation --- */

/* put, then update the 64-bit signal word `sig_addr`@pe (symmetric) with `signal`
 * (ISHMEM_SIGNAL_SET / _ADD); the update becomes visible only after the payload. */
int ishmem_putmem_signal(int my_pe, void *dest, const void *src, size_t nbytes,
                         uint64_t *sig_addr, uint64_t signal, int sig_op, int pe);
/* Enqueues a bounded device-side wait on my_pe's stream until `*ivar`@my_pe cmp value.
 * On expiry the status word latches ISHMEM_ERR_TIMEOUT and the stream continues. */
int ishmem_uint64_wait_until(int my_pe, uint64_t *ivar, int cmp, uint64_t value);
/* One evaluation of the comparison on my_pe's copy of `ivar`, after everything already
 * enqueued on my_pe's stream: HOST *result = 1 or 0.  Blocks the host. */
int ishmem_uint64_test(int my_pe, uint64_t *ivar, int cmp, uint64_t value, int *result);
/* Waits on `nelems` (at most 256) consecutive symmetric 64-bit words of my_pe (OpenSHMEM 1.5
 * wait_until_all / _any / _some), bounded like ishmem_uint64_wait_until.  `status` is the
 * standard's mask: a DEVICE array of nelems ints (or NULL) -- words whose entry is non-zero are
 * left out.  _all is stream-ordered.  _any writes the index of a satisfied word to HOST *index;
 * _some waits for at least one and writes the ascending indices of all words satisfied at that
 * moment to HOST indices[0..*count-1] (room for nelems).  _any and _some block the host and
 * return ISHMEM_ERR_TIMEOUT when the wait gave up. */
int ishmem_uint64_wait_until_all(int my_pe, uint64_t *ivars, size_t nelems, const int *status, int cmp,
                                 uint64_t value);
int ishmem_uint64_wait_until_any(int my_pe, uint64_t *ivars, size_t nelems, const int *status, int cmp,
                                 uint64_t value, size_t *index);
int ishmem_uint64_wait_until_some(int my_pe, uint64_t *ivars, size_t nelems, size_t *indices, const int *status,
                                  int cmp, uint64_t value, size_t *count);
/* fence: orders my_pe's earlier puts before its later ones per target (stream order
 * already gives this; kept for API parity).  quiet: completes all outstanding operations
 * of my_pe, including _nbi transfers on the copy engine, in stream order. */
int ishmem_fence(int my_pe);
int ishmem_quiet(int my_pe);
/* sync: team members wait for one another (Section 3.7.2: each PE sends an atomic
 * increment to every other member's counter and waits on its own).  Runs the push
 * algorithm in one co-resident launch.  barrier_all = quiet on every PE + sync, and blocks
 * the host until done.  sync_all = team_sync(WORLD), stream-ordered. */
int ishmem_team_sync(ishmem_team_t team);
int ishmem_sync_all(void);
int ishmem_barrier_all(void);
/* Strided sub-team of a parent team; returns the new team or ISHMEM_TEAM_INVALID. */
ishmem_team_t ishmem_team_split_strided(ishmem_team_t parent, int start, int stride, int size);
/* 2-D split (OpenSHMEM 1.5 team_split_2d): the parent's members are laid out row-major with
 * `xrange` columns; *xaxis_team receives the team of parent member `parent_index`'s row (stride 1)
 * and *yaxis_team that of its column (stride xrange).  Each call creates two new teams (destroy
 * them with ishmem_team_destroy).  ISHMEM_ERR_ARG when an argument is invalid or the team table
 * is full (in which case nothing is created). */
int ishmem_team_split_2d(ishmem_team_t parent, int xrange, int parent_index, ishmem_team_t *xaxis_team,
                         ishmem_team_t *yaxis_team);
int ishmem_team_destroy(ishmem_team_t team);
int ishmem_team_n_pes(ishmem_team_t team);
/* Index of world PE `pe` inside `team`, or -1 when it is not a member (OpenSHMEM's team_my_pe, with
 * the PE explicit because all PEs live in this process). */
int ishmem_team_my_pe(ishmem_team_t team, int pe);
/* The PE with index `src_pe` in src_team, expressed as an index in dest_team; -1 when it is not
 * a member of dest_team or an argument is invalid. */
int ishmem_team_translate_pe(ishmem_team_t src_team, int src_pe, ishmem_team_t dest_team);
/* Library identification (OpenSHMEM info routines): the OpenSHMEM level the API follows, and a
 * name of at most ISHMEM_MAX_NAME_LEN - 1 characters copied to HOST `name`. */
#define ISHMEM_MAJOR_VERSION 1
#define ISHMEM_MINOR_VERSION 5
#define ISHMEM_MAX_NAME_LEN 64
void ishmem_info_get_version(int *major, int *minor);
void ishmem_info_get_name(char *name);

/* --------------------------------------------------------------- remote atomics --- */

/* One atomic on the integer at symmetric address `target` on PE `pe`, issued by my_pe.
 * Non-fetching forms are stream-ordered; fetching forms block the host and write the old
 * value to HOST memory `fetched_host`. */
#define ISHMEM_DECL_AMO(NAME, T)                                                               \
    int ishmem_##NAME##_atomic_add(int my_pe, T *target, T value, int pe);                     \
    int ishmem_##NAME##_atomic_inc(int my_pe, T *target, int pe);                              \
    int ishmem_##NAME##_atomic_set(int my_pe, T *target, T value, int pe);                     \
    int ishmem_##NAME##_atomic_and(int my_pe, T *target, T value, int pe);                     \
    int ishmem_##NAME##_atomic_or(int my_pe, T *target, T value, int pe);                      \
    int ishmem_##NAME##_atomic_xor(int my_pe, T *target, T value, int pe);                     \
    int ishmem_##NAME##_atomic_fetch(int my_pe, T *fetched_host, const T *target, int pe);     \
    int ishmem_##NAME##_atomic_fetch_add(int my_pe, T *fetched_host, T *target, T value, int pe); \
    int ishmem_##NAME##_atomic_fetch_inc(int my_pe, T *fetched_host, T *target, int pe);       \
    int ishmem_##NAME##_atomic_swap(int my_pe, T *fetched_host, T *target, T value, int pe);   \
    int ishmem_##NAME##_atomic_compare_swap(int my_pe, T *fetched_host, T *target, T cond,     \
                                            T value, int pe);                                  \
    int ishmem_##NAME##_atomic_fetch_and(int my_pe, T *fetched_host, T *target, T value, int pe); \
    int ishmem_##NAME##_atomic_fetch_or(int my_pe, T *fetched_host, T *target, T value, int pe);  \
    int ishmem_##NAME##_atomic_fetch_xor(int my_pe, T *fetched_host, T *target, T value, int pe);
ISHMEM_DECL_AMO(int32, int32_t)
ISHMEM_DECL_AMO(int64, int64_t)
ISHMEM_DECL_AMO(uint32, uint32_t)
ISHMEM_DECL_AMO(uint64, uint64_t)
#undef ISHMEM_DECL_AMO

/* Device-initiated batches (one op per GPU thread, every thread of the launch issuing): op i is
 * issued by PE (i mod npes); word w of the table lives on PE (w mod npes) at
 * table + 8*(w div npes).  word_idx/inc/cond/value/fetched are device arrays of `nops`
 * entries (fetched may be NULL).  aggregate = 0: one atomic per op.  aggregate = 1: the lanes
 * of a warp that hit the same word combine into one atomic.  aggregate = 2: the ops of a whole
 * block (8 per thread) that hit the same word combine in shared-memory accumulators (2048
 * direct-mapped slots; ops whose slot is taken by another word go to the table directly) and
 * one atomic per used slot reaches the table.  In every mode each op's fetched value is the one
 * it would have seen in one valid serialisation, and the final table is the same.  One launch
 * on the team stream. */
int ishmemx_int64_atomic_fetch_add_batch(int64_t *table, const int32_t *word_idx,
                                         const int64_t *inc, int64_t *fetched, size_t nops,
                                         int threads, int aggregate);
/* compare_swap: aggregate = 1 lets the lanes of a warp that hit the same word act as one group
 * whose operations are applied back to back in lane order by a single compare-and-swap of the
 * word (a read alone when the group changes nothing); aggregate = 0: one atomic per op. */
int ishmemx_int64_atomic_compare_swap_batch(int64_t *table, const int32_t *word_idx,
                                            const int64_t *cond, const int64_t *value,
                                            int64_t *fetched, size_t nops, int threads, int aggregate);

/* ------------------------------------------------- collectives (Section 3.7.2) --- */

/* broadcast: dest@q[0:nbytes] = src@root for every team member q ("push": the root stores
 * into every destination, destinations in the inner loop).  `root` is the index inside
 * the team.  The root's own dest is written too unless ishmemx_set_bcast_root_dest(0). */
int ishmem_broadcastmem(ishmem_team_t team, void *dest, const void *src, size_t nbytes, int root);
int ishmemx_set_bcast_root_dest(int enable);
/* fcollect: dest@q[i*nbytes:(i+1)*nbytes] = src@member_i for every member q (allgather
 * with equal contributions; push). */
int ishmem_fcollectmem(ishmem_team_t team, void *dest, const void *src, size_t nbytes);
/* collect: fcollect with contributions of different sizes ("collect (which is like MPI
 * allgather)", Section 3.7.2): every member's dest becomes the concatenation, in team order, of
 * the members' sources; member i contributes nbytes_per_member[i] bytes (HOST array of team-size
 * entries -- all PEs live in this process, so the sizes need no exchange).  Push. */
int ishmem_collectmem(ishmem_team_t team, void *dest, const void *src, const size_t *nbytes_per_member);
/* alltoall (OpenSHMEM 1.5): dest@q[i*nbytes + k] = src@member_i[q*nbytes + k]: block q of member
 * i's source lands in block i of member q's dest.  dest and src must not overlap.  Push. */
int ishmem_alltoallmem(ishmem_team_t team, void *dest, const void *src, size_t nbytes);
/* Typed names of the four data-movement collectives (counts in elements; addresses aligned to
 * the element). */
#define ISHMEM_DECL_COLL(NAME, T)                                                                          \
    int ishmem_##NAME##_broadcast(ishmem_team_t team, T *dest, const T *src, size_t nelems, int root);      \
    int ishmem_##NAME##_fcollect(ishmem_team_t team, T *dest, const T *src, size_t nelems);                 \
    int ishmem_##NAME##_collect(ishmem_team_t team, T *dest, const T *src, const size_t *nelems_per_member); \
    int ishmem_##NAME##_alltoall(ishmem_team_t team, T *dest, const T *src, size_t nelems);
ISHMEM_DECL_COLL(float, float)
ISHMEM_DECL_COLL(double, double)
ISHMEM_DECL_COLL(int, int)
ISHMEM_DECL_COLL(long, long)
ISHMEM_DECL_COLL(int32, int32_t)
ISHMEM_DECL_COLL(int64, int64_t)
ISHMEM_DECL_COLL(uint8, uint8_t)
ISHMEM_DECL_COLL(uint32, uint32_t)
ISHMEM_DECL_COLL(uint64, uint64_t)
#undef ISHMEM_DECL_COLL
/* reduce: dest@q[j] = ((src@m0[j] op src@m1[j]) op ...) op src@m_{P-1}[j], folded in team
 * order (floating point bit-exact in that order), for every member q.  dest and src may
 * not overlap unless identical, which is handled with snapshot semantics only by the
 * SPLIT algorithm.  Integer sum/prod wrap. */
int ishmemx_reduce(ishmem_team_t team, void *dest, const void *src, size_t nreduce, int op,
                   int dtype, int algorithm);
#define ISHMEM_DECL_REDUCE(NAME, T, OP)                                                        \
    int ishmem_##NAME##_##OP##_reduce(ishmem_team_t team, T *dest, const T *src, size_t nreduce);
#define ISHMEM_DECL_REDUCE_ARITH(NAME, T)                                                      \
    ISHMEM_DECL_REDUCE(NAME, T, sum) ISHMEM_DECL_REDUCE(NAME, T, max)                          \
    ISHMEM_DECL_REDUCE(NAME, T, min) ISHMEM_DECL_REDUCE(NAME, T, prod)
#define ISHMEM_DECL_REDUCE_BITS(NAME, T)                                                       \
    ISHMEM_DECL_REDUCE(NAME, T, and) ISHMEM_DECL_REDUCE(NAME, T, or) ISHMEM_DECL_REDUCE(NAME, T, xor)
ISHMEM_DECL_REDUCE_ARITH(int32, int32_t)
ISHMEM_DECL_REDUCE_ARITH(int64, int64_t)
ISHMEM_DECL_REDUCE_ARITH(uint32, uint32_t)
ISHMEM_DECL_REDUCE_ARITH(uint64, uint64_t)
ISHMEM_DECL_REDUCE_ARITH(float, float)
ISHMEM_DECL_REDUCE_ARITH(double, double)
ISHMEM_DECL_REDUCE_BITS(int32, int32_t)
ISHMEM_DECL_REDUCE_BITS(int64, int64_t)
ISHMEM_DECL_REDUCE_BITS(uint32, uint32_t)
ISHMEM_DECL_REDUCE_BITS(uint64, uint64_t)
/* Integer types of 8 to 64 bits (Section 3.7.2): sum and product modulo 2^8 / 2^16 */
ISHMEM_DECL_REDUCE_ARITH(int8, int8_t)
ISHMEM_DECL_REDUCE_ARITH(uint8, uint8_t)
ISHMEM_DECL_REDUCE_ARITH(int16, int16_t)
ISHMEM_DECL_REDUCE_ARITH(uint16, uint16_t)
ISHMEM_DECL_REDUCE_BITS(int8, int8_t)
ISHMEM_DECL_REDUCE_BITS(uint8, uint8_t)
ISHMEM_DECL_REDUCE_BITS(int16, int16_t)
ISHMEM_DECL_REDUCE_BITS(uint16, uint16_t)
#undef ISHMEM_DECL_REDUCE
#undef ISHMEM_DECL_REDUCE_ARITH
#undef ISHMEM_DECL_REDUCE_BITS
/* Launch geometry of collective kernels: blocks per PE (0 = automatic) and threads. */
int ishmemx_set_collective_geometry(int groups_per_pe, int threads);

/* Device-resident collectives: ONE co-resident launch in which one work-group per PE calls
 * the device routine ishmemx_{broadcastmem,fcollectmem,reduce,sync_all}_work_group of
 * ishmem_device.cuh, with in-kernel push synchronisation (for tests and latency
 * measurements of the device API itself).  which: 0 broadcast, 1 fcollect, 2 reduce
 * (op/dtype as above), 3 sync_all, 4 alltoall, 5 collect with the sizes exchanged inside the
 * kernel (member i contributes n * ((i mod 3) + 1) / 3 bytes); the call is repeated `repeat`
 * times. */
int ishmemx_collective_on_device(int which, ishmem_team_t team, void *dest, const void *src,
                                 size_t n, int root, int op, int dtype, int threads, int repeat);

/* ----------------------------------------------- device-initiated test programs --- */

/* put_signal / wait_until ping-pong between PE a and PE b, entirely inside one
 * co-resident launch: `rounds` round trips of `nbytes` (work-group put_signal with
 * `threads` threads, SIGNAL_SET to the round number, wait_until GE).  data: symmetric,
 * >= nbytes; sig: symmetric 64-bit word, zero on entry.  Writes the mean half round trip
 * in nanoseconds (measured in-kernel with the global timer) to HOST memory `half_rtt_ns`.
 * Each round stamps the round number into the first and last 8 bytes of the payload; the
 * receiver counts stamps that do not match the signalled round into HOST `mismatches`
 * (a non-zero count means a signal overtook its payload).  Blocks the host. */
int ishmemx_pingpong(int pe_a, int pe_b, void *data, uint64_t *sig, size_t nbytes, int rounds,
                     int threads, double *half_rtt_ns, uint64_t *mismatches);

/* Where a half round trip of that exchange goes.  The same ping-pong with the put_signal written out
 * phase by phase and the SM cycle counter read between the phases by the first thread of each side
 * (`rounds` rounds, `threads` threads per side; sig: 4 symmetric words, zero on entry; staged != 0: the
 * kernel reads its context from a copy in shared memory, as k_pingpong does, 0: from global memory).
 * Writes 14 doubles to HOST `ns_out`, nanoseconds per round at the device's nominal SM clock:
 *   [0..4]  side A: wait for the answer / address translation / copy / block barrier / release of the
 *           signal word (fence + store); a phase includes the wait for the loads its first instruction
 *           needs, so the five add up to A's round;
 *   [5..9]  side B, the same;
 *   [10]    one dependent relaxed load of a word in L2 (one trip), [11] a store followed by
 *           st.release.gpu, [12] st.release.gpu with nothing pending;
 *   [13]    half round trip by the global timer.
 * Blocks the host.  Errors as ishmemx_pingpong. */
int ishmemx_pingpong_phases(int pe_a, int pe_b, void *data, uint64_t *sig, size_t nbytes, int rounds,
                            int threads, int staged, double *ns_out);

/* Device-initiated latency of one collaboration level (the measurement method of Section 4:
 * many back-to-back operations inside one kernel, timed on the device).  ONE work-group of
 * `threads` threads runs as PE my_pe and issues `iters` puts (is_get = 0) or gets of `nbytes`
 * to/from PE `pe`, each followed by quiet: by its first thread alone (ISHMEMX_WORK_ITEM), by
 * its first warp (ISHMEMX_SUB_GROUP), or by all threads (ISHMEMX_WORK_GROUP, _BULK, _ENGINE).  dest/src
 * as for ishmem_putmem / ishmem_getmem.  Writes the mean time per operation in nanoseconds
 * (global timer, read inside the kernel) to HOST memory `ns_per_op`.  Blocks the host. */
int ishmemx_rma_latency(int my_pe, void *dest, const void *src, size_t nbytes, int pe, int is_get,
                        int level, int threads, int iters, double *ns_per_op);

/* Overlap workload: `iters` sweeps of the 5-point Jacobi update on an ny x nx float64
 * grid cut into npes row strips (the first ny mod npes strips have one more row): each sweep
 * every PE sends its first and last rows to the neighbours' halo rows with in-kernel work-group
 * put_signal, updates its interior rows meanwhile, and updates its edge rows once its own halos
 * have arrived.  buf0/buf1:
 * symmetric, (ceil(ny/npes)+2)*nx doubles each, strip row r at local row r+1 of buf0 on entry
 * (buf1 is overwritten); sig: symmetric, 4 words, zero on entry.  overlap = 0 disables the
 * interior-first ordering (exchange, wait, then compute).
 * threads = 0 (and an even nx): the library shapes the launches itself -- many short launches whose
 * first blocks send the halo rows (in-kernel work-group put_signal) and whose other blocks each
 * take a band of rows of a few neighbouring column tiles, one warp per tile, numbered so that the
 * blocks sweep the grid in launch order; only the bands at the two ends of a strip wait for a halo,
 * the interior never does.  A launch does up to SIX sweeps: a warp's register window carries that
 * many time levels, every element is read once and the last level written once, and as many halo
 * rows go each way as the launch does sweeps -- the first into the halo row of the buffer being
 * read, the second into the halo row of the buffer being written, the third to sixth into up to
 * eight rows per PE that the call takes from the symmetric heap and gives back (2 * (k - 2) * nx * 8
 * bytes for launches of k sweeps; when the heap has no room for them the call stays at four, else
 * at two sweeps per launch).  The result of every cell is the same expression in the same order
 * as in single sweeps, bit for bit.  The sweeps are cut into launches of 6 .. 1 so that the number
 * of launches has the parity of iters (each launch moves the grid to the other buffer) at the
 * least cost by a table of measured launch times; a strip must own as many rows as a launch does
 * sweeps.  At 16384^2 on 12 PEs: 160 us per sweep with six sweeps per launch, 170 with five, 185
 * with four, 240 with three, 345 with two, 640 with one (the copy rate).  With residual_sq_host
 * NULL the last launch forms no residual and runs like the others.
 * ISHMEMX_OPT_JACOBI_FUSE caps the sweeps per launch (0 = always one), ISHMEMX_OPT_JACOBI_WIDE
 * picks two or four columns per lane (ishmemx_set_option).  groups_per_pe is not used by this
 * form and nothing needs to be co-resident.
 * threads > 0 (a multiple of 32 up to 1024): one persistent co-resident launch of
 * npes x groups_per_pe blocks of that size for all sweeps; the blocks of a PE take bands of rows,
 * one of them sends each halo row, and neighbouring blocks hand over through flags.
 * ISHMEM_ERR_NOT_CORESIDENT when the blocks cannot all be resident at once.  The option
 * ISHMEMX_OPT_JACOBI_SPLIT = 1 (rows) | 2 (columns) selects the persistent kernel also for threads = 0,
 * with the strips cut by rows, or by ranges of column tiles (one warp per tile; every block then
 * sends its columns of the halo rows); groups_per_pe is clamped to the rows (tiles) of the
 * shortest strip.
 * The final strips are in buf0 if iters is even, else buf1.  residual_sq_host (HOST, may be
 * NULL) receives ||u_iters - u_(iters-1)||_2^2 over the interior.  Blocks the host. */
int ishmemx_jacobi(double *buf0, double *buf1, uint64_t *sig, size_t ny, size_t nx, int iters,
                   int overlap, int groups_per_pe, int threads, double *residual_sq_host);

/* How ishmemx_jacobi cuts `iters` sweeps into launches when a launch may do up to max_depth (1..6)
 * sweeps: writes the sweeps of each launch, deepest first, to HOST depths_out (room for `capacity`
 * entries; may be NULL with capacity 0) and returns the number of launches, which always has the
 * parity of iters (every launch moves the grid to the other buffer), or ISHMEM_ERR_ARG.  Pure host
 * arithmetic: needs neither a device nor ishmem_init. */
int ishmemx_jacobi_launch_depths(int iters, int max_depth, int *depths_out, int capacity);

/* The same Jacobi program for callers that must not allocate device memory at the point of
 * the call -- a frozen memory pool, a loop where cudaMalloc's device-wide synchronisation is
 * not acceptable, an allocator that owns the whole GPU.  (The paper has no counterpart; this
 * is a convenience of this library.)  The kernel's scratch -- one sweep counter and one
 * residual partial per block -- sits in a fixed 32 KiB device array inside the library, which
 * every GPU that loads the library holds until the process exits; the call itself performs no
 * cudaMalloc/cudaFree and calls no allocating routine.  Limits and caveats:
 *   - npes * groups_per_pe (after clamping groups_per_pe to the shortest strip) must not
 *     exceed 2048 blocks; larger launches are refused with ISHMEM_ERR_ARG and
 *     ishmemx_last_cuda_error() names the limit.
 *   - The first call on each device resolves the array's device address
 *     (cudaGetSymbolAddress); make that first call before any stream capture begins, and from
 *     one host thread: the per-device address cache is filled without a lock (two threads
 *     racing there would store the same value, but the call is not documented as re-entrant).
 *   - All calls share the one array.  It still holds the previous call's contents, so each
 *     call clears the part it uses first; two calls whose kernels overlap on the GPU (from
 *     two host threads, say) would race on it -- serialise them.
 *   - It always runs the persistent kernel (threads = 0: strips cut by column tiles when the grid
 *     is wide enough, else by rows with 512 threads); the one-launch-per-sweep form keeps one
 *     residual term per tile block and does not fit the fixed array.
 * Arguments, results and error codes are otherwise those of ishmemx_jacobi. */
int ishmemx_jacobi_noalloc(double *buf0, double *buf1, uint64_t *sig, size_t ny, size_t nx, int iters,
                           int overlap, int groups_per_pe, int threads, double *residual_sq_host);

/* Host-buffer convenience for end-to-end measurements: for every PE p, copy `nbytes` from HOST
 * `src_host` (per-PE stride `nbytes`) into src@p, let PE p put it to dest@((p + shift) mod npes)
 * (device call of the given level with `groups` work-groups of `threads` threads; groups == 0: one
 * tile of threads x 128 bytes per work-group), and copy that
 * destination back to HOST `dest_host` (same layout).  Each PE's three steps run on its own
 * stream, so transfers in the two directions overlap between PEs; with pinned host memory the
 * copies are asynchronous.  Blocks the host until everything has arrived. */
int ishmemx_host_put_ring(void *dest_host, const void *src_host, void *dest, void *src,
                          size_t nbytes, int shift, int level, int threads, int groups);

#ifdef __cplusplus
}
#endif
#endif /* ISHMEM_H */
