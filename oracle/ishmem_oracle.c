/*
 * ishmem_oracle.c -- plain, sequential CPU model of the OpenSHMEM semantics that
 * Intel SHMEM implements (arXiv 2409.20476).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It exists so that the CUDA
 * library's results can be compared with an independent, obviously-correct
 * statement of what each operation computes.  Only tests, the smoke check and
 * the benchmark's cpu_baseline/reference legs may call it.  It shares no code,
 * header, table or helper with the CUDA path and knows nothing about it.
 *
 * Model: `npes` processing elements (PEs), each owning one byte array of
 * `heap_bytes` (its symmetric heap).  A symmetric object is named by its byte
 * offset inside the heap: the layout is identical on every PE, the contents are
 * not (Section 2.3, "OpenSHMEM Memory and Execution Model").  Every operation
 * is applied at once, in program order, by one thread; there is no blocking,
 * no vectorisation, no reordering.  Where an operation has a plain definition
 * (copy, fold, read-modify-write) the function below is that definition.
 *
 * Parity pins (tests/test_oracle_*.py): put/get against Python's byte-at-a-time
 * model on tiny heaps, closed forms of PE-indexed patterns for reduce /
 * fcollect / broadcast, numpy wrap-around sums (also for 8- and 16-bit elements), numpy strided
 * slices for iput / iget, np.concatenate for collect, a block transpose for alltoall (with its
 * involution property), conservation and chain checks
 * for atomics, hand-worked allocator offsets, the truth table of oracle_test,
 * Jacobi eigenmode decay, decomposition independence and a hand case that fixes
 * the association order of the update.
 * "parity unpinned": the root-writes-dest reading of broadcast (the OpenSHMEM
 * text is not at hand; both readings are offered and tested).
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC
 */
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_INVALID_PE (-1)
#define ORACLE_ERR_NOT_SYMMETRIC (-2)
#define ORACLE_ERR_ALIGN (-3)
#define ORACLE_ERR_OOM (-4)
#define ORACLE_ERR_ARG (-5)

/* element types of typed operations */
enum { T_INT32 = 0, T_INT64 = 1, T_FLOAT = 2, T_DOUBLE = 3, T_UINT32 = 4, T_UINT64 = 5,
       T_INT8 = 6, T_UINT8 = 7, T_INT16 = 8, T_UINT16 = 9 };
/* reduction operators (Section 3.7.2, "Reduction": min, max, sum, product, and/or/xor) */
enum { R_SUM = 0, R_MAX = 1, R_MIN = 2, R_PROD = 3, R_AND = 4, R_OR = 5, R_XOR = 6 };
/* atomic operations */
enum {
    A_FETCH_ADD = 0, A_ADD = 1, A_FETCH_INC = 2, A_INC = 3, A_FETCH = 4, A_SET = 5,
    A_SWAP = 6, A_COMPARE_SWAP = 7, A_FETCH_AND = 8, A_FETCH_OR = 9, A_FETCH_XOR = 10
};
/* signal operators and wait_until comparisons */
enum { SIG_SET = 0, SIG_ADD = 1 };
enum { C_EQ = 0, C_NE = 1, C_GT = 2, C_GE = 3, C_LT = 4, C_LE = 5 };

typedef struct oracle {
    int npes;
    size_t heap_bytes;
    unsigned char **heap; /* heap[pe] = that PE's symmetric heap */
    size_t brk;           /* bump allocator cursor (same on every PE) */
} oracle_t;

static size_t type_size(int t)
{
    switch (t) {
    case T_INT32: case T_FLOAT: case T_UINT32: return 4;
    case T_INT64: case T_DOUBLE: case T_UINT64: return 8;
    case T_INT8: case T_UINT8: return 1;
    case T_INT16: case T_UINT16: return 2;
    default: return 0;
    }
}

oracle_t *oracle_create(int npes, size_t heap_bytes)
{
    if (npes < 1) return NULL;
    oracle_t *o = (oracle_t *)calloc(1, sizeof(*o));
    if (!o) return NULL;
    o->npes = npes;
    o->heap_bytes = heap_bytes;
    o->heap = (unsigned char **)calloc((size_t)npes, sizeof(unsigned char *));
    if (!o->heap) { free(o); return NULL; }
    for (int p = 0; p < npes; ++p) {
        o->heap[p] = (unsigned char *)calloc(heap_bytes ? heap_bytes : 1, 1);
        if (!o->heap[p]) {
            for (int q = 0; q < p; ++q) free(o->heap[q]);
            free(o->heap); free(o);
            return NULL;
        }
    }
    return o;
}

void oracle_destroy(oracle_t *o)
{
    if (!o) return;
    for (int p = 0; p < o->npes; ++p) free(o->heap[p]);
    free(o->heap);
    free(o);
}

int oracle_n_pes(const oracle_t *o) { return o->npes; }
size_t oracle_heap_bytes(const oracle_t *o) { return o->heap_bytes; }

/* Address translation (Section 3.7.1): the object at offset `off` on PE `pe`
 * lives at that PE's heap base plus the same offset.  NULL when the PE does
 * not exist or the range [off, off+n) leaves the heap. */
void *oracle_ptr(const oracle_t *o, size_t off, size_t n, int pe)
{
    if (pe < 0 || pe >= o->npes) return NULL;
    if (off > o->heap_bytes || n > o->heap_bytes - off) return NULL;
    return o->heap[pe] + off;
}

static int check(const oracle_t *o, size_t off, size_t n, int pe)
{
    if (pe < 0 || pe >= o->npes) return ORACLE_ERR_INVALID_PE;
    if (off > o->heap_bytes || n > o->heap_bytes - off) return ORACLE_ERR_NOT_SYMMETRIC;
    return ORACLE_OK;
}

/* Symmetric allocation: the same offset on every PE (Section 2.3).  A bump
 * cursor is all the model needs; `align` must be a power of two. */
int oracle_malloc(oracle_t *o, size_t size, size_t align, size_t *off_out)
{
    if (align == 0 || (align & (align - 1))) return ORACLE_ERR_ALIGN;
    size_t start = (o->brk + align - 1) & ~(align - 1);
    if (start > o->heap_bytes || size > o->heap_bytes - start) return ORACLE_ERR_OOM;
    o->brk = start + size;
    *off_out = start;
    return ORACLE_OK;
}

void oracle_reset_allocator(oracle_t *o) { o->brk = 0; }

/* ---- RMA (Section 3.7.1) ------------------------------------------------ */

/* put: PE `my_pe` copies n bytes from its own address `src` (any memory it can
 * read) to the symmetric object at `dest_off` on PE `pe`. */
int oracle_putmem(oracle_t *o, int my_pe, size_t dest_off, const void *src, size_t n, int pe)
{
    int rc = check(o, 0, 0, my_pe);
    if (rc) return rc;
    rc = check(o, dest_off, n, pe);
    if (rc) return rc;
    const unsigned char *s = (const unsigned char *)src;
    unsigned char *d = o->heap[pe] + dest_off;
    for (size_t i = 0; i < n; ++i) d[i] = s[i];
    return ORACLE_OK;
}

/* get: PE `my_pe` copies n bytes from the symmetric object at `src_off` on PE
 * `pe` to its own address `dest`. */
int oracle_getmem(oracle_t *o, int my_pe, void *dest, size_t src_off, size_t n, int pe)
{
    int rc = check(o, 0, 0, my_pe);
    if (rc) return rc;
    rc = check(o, src_off, n, pe);
    if (rc) return rc;
    const unsigned char *s = o->heap[pe] + src_off;
    unsigned char *d = (unsigned char *)dest;
    for (size_t i = 0; i < n; ++i) d[i] = s[i];
    return ORACLE_OK;
}

/* strided put (OpenSHMEM iput; the strided form of put that Section 3.7.1 lists): element k
 * of the source, taken every `sst` elements from `src`, becomes element k*dst of the symmetric
 * object at `dest_off` on PE `pe`, k = 0..nelems-1.  Elements are `esize` bytes; strides are in
 * elements and at least 1. */
int oracle_iput(oracle_t *o, int my_pe, size_t dest_off, const void *src, size_t dst, size_t sst,
                size_t nelems, size_t esize, int pe)
{
    int rc = check(o, 0, 0, my_pe);
    if (rc) return rc;
    if (dst < 1 || sst < 1 || esize < 1) return ORACLE_ERR_ARG;
    if (nelems) {
        if ((nelems - 1) > (o->heap_bytes / esize) / dst) return ORACLE_ERR_NOT_SYMMETRIC;
        rc = check(o, dest_off, ((nelems - 1) * dst + 1) * esize, pe);
        if (rc) return rc;
    } else if ((rc = check(o, dest_off, 0, pe))) {
        return rc;
    }
    const unsigned char *s = (const unsigned char *)src;
    unsigned char *d = o->heap[pe] + dest_off;
    for (size_t k = 0; k < nelems; ++k)
        for (size_t b = 0; b < esize; ++b) d[k * dst * esize + b] = s[k * sst * esize + b];
    return ORACLE_OK;
}

/* strided get (iget): element k*sst of the symmetric object at `src_off` on PE `pe` becomes
 * element k*dst of the caller's `dest`. */
int oracle_iget(oracle_t *o, int my_pe, void *dest, size_t src_off, size_t dst, size_t sst,
                size_t nelems, size_t esize, int pe)
{
    int rc = check(o, 0, 0, my_pe);
    if (rc) return rc;
    if (dst < 1 || sst < 1 || esize < 1) return ORACLE_ERR_ARG;
    if (nelems) {
        if ((nelems - 1) > (o->heap_bytes / esize) / sst) return ORACLE_ERR_NOT_SYMMETRIC;
        rc = check(o, src_off, ((nelems - 1) * sst + 1) * esize, pe);
        if (rc) return rc;
    } else if ((rc = check(o, src_off, 0, pe))) {
        return rc;
    }
    const unsigned char *s = o->heap[pe] + src_off;
    unsigned char *d = (unsigned char *)dest;
    for (size_t k = 0; k < nelems; ++k)
        for (size_t b = 0; b < esize; ++b) d[k * dst * esize + b] = s[k * sst * esize + b];
    return ORACLE_OK;
}

/* scalar p / g: one element of `esize` bytes (the ishmem_long_p walk-through of
 * Section 3.7.1).  The element must be naturally aligned. */
int oracle_p(oracle_t *o, size_t dest_off, const void *value, size_t esize, int pe)
{
    if (esize == 0 || dest_off % esize) return ORACLE_ERR_ALIGN;
    return oracle_putmem(o, pe, dest_off, value, esize, pe);
}

int oracle_g(oracle_t *o, void *value_out, size_t src_off, size_t esize, int pe)
{
    if (esize == 0 || src_off % esize) return ORACLE_ERR_ALIGN;
    return oracle_getmem(o, pe, value_out, src_off, esize, pe);
}

/* ---- signalling and point-to-point synchronisation ----------------------- */

/* put_signal: the payload is delivered first, then the 64-bit signal word at
 * `sig_off` on the target is set to, or incremented by, `signal`. */
int oracle_putmem_signal(oracle_t *o, int my_pe, size_t dest_off, const void *src, size_t n,
                         size_t sig_off, uint64_t signal, int sig_op, int pe)
{
    if (sig_off % 8) return ORACLE_ERR_ALIGN;
    int rc = check(o, sig_off, 8, pe);
    if (rc) return rc;
    rc = oracle_putmem(o, my_pe, dest_off, src, n, pe);
    if (rc) return rc;
    uint64_t *sig = (uint64_t *)(o->heap[pe] + sig_off);
    if (sig_op == SIG_SET) *sig = signal;
    else if (sig_op == SIG_ADD) *sig = *sig + signal;
    else return ORACLE_ERR_ARG;
    return ORACLE_OK;
}

/* The comparison wait_until blocks on.  In a sequential schedule nothing can
 * block: 1 = the condition holds (wait_until would return), 0 = it would block,
 * negative = error. */
int oracle_test(const oracle_t *o, int my_pe, size_t ivar_off, int cmp, uint64_t value)
{
    if (ivar_off % 8) return ORACLE_ERR_ALIGN;
    int rc = check(o, ivar_off, 8, my_pe);
    if (rc) return rc;
    uint64_t v = *(const uint64_t *)(o->heap[my_pe] + ivar_off);
    switch (cmp) {
    case C_EQ: return v == value;
    case C_NE: return v != value;
    case C_GT: return v > value;
    case C_GE: return v >= value;
    case C_LT: return v < value;
    case C_LE: return v <= value;
    default: return ORACLE_ERR_ARG;
    }
}

/* ---- atomic memory operations -------------------------------------------- */

/* One read-modify-write on the 32- or 64-bit integer at `target_off` on PE
 * `pe`.  Arithmetic wraps modulo 2^width (computed unsigned).  `*fetched`
 * receives the value before the operation (for every op; callers of
 * non-fetching ops ignore it). */
int oracle_atomic(oracle_t *o, int op, int width_bytes, size_t target_off, uint64_t operand,
                  uint64_t cond, int pe, uint64_t *fetched)
{
    if (width_bytes != 4 && width_bytes != 8) return ORACLE_ERR_ARG;
    if (target_off % (size_t)width_bytes) return ORACLE_ERR_ALIGN;
    int rc = check(o, target_off, (size_t)width_bytes, pe);
    if (rc) return rc;
    unsigned char *t = o->heap[pe] + target_off;
    uint64_t old;
    if (width_bytes == 8) old = *(uint64_t *)t;
    else old = *(uint32_t *)t;
    uint64_t neu = old;
    switch (op) {
    case A_FETCH_ADD: case A_ADD: neu = old + operand; break;
    case A_FETCH_INC: case A_INC: neu = old + 1; break;
    case A_FETCH: neu = old; break;
    case A_SET: case A_SWAP: neu = operand; break;
    case A_COMPARE_SWAP:
        if (width_bytes == 4) { if ((uint32_t)old == (uint32_t)cond) neu = operand; }
        else if (old == cond) neu = operand;
        break;
    case A_FETCH_AND: neu = old & operand; break;
    case A_FETCH_OR: neu = old | operand; break;
    case A_FETCH_XOR: neu = old ^ operand; break;
    default: return ORACLE_ERR_ARG;
    }
    if (width_bytes == 8) *(uint64_t *)t = neu;
    else *(uint32_t *)t = (uint32_t)neu;
    if (fetched) *fetched = old;
    return ORACLE_OK;
}

/* Batch of 64-bit fetch_add operations applied in index order.  Word w of the
 * table lives on PE (w mod npes) at offset table_off + 8*(w div npes). */
int oracle_int64_fetch_add_batch(oracle_t *o, size_t table_off, const int32_t *word,
                                 const int64_t *inc, int64_t *fetched, size_t nops)
{
    for (size_t i = 0; i < nops; ++i) {
        if (word[i] < 0) return ORACLE_ERR_ARG;
        int pe = word[i] % o->npes;
        size_t off = table_off + 8 * (size_t)(word[i] / o->npes);
        uint64_t old;
        int rc = oracle_atomic(o, A_FETCH_ADD, 8, off, (uint64_t)inc[i], 0, pe, &old);
        if (rc) return rc;
        if (fetched) fetched[i] = (int64_t)old;
    }
    return ORACLE_OK;
}

/* Batch of 64-bit compare_swap operations applied in index order, same word
 * placement as above. */
int oracle_int64_compare_swap_batch(oracle_t *o, size_t table_off, const int32_t *word,
                                    const int64_t *cond, const int64_t *value, int64_t *fetched,
                                    size_t nops)
{
    for (size_t i = 0; i < nops; ++i) {
        if (word[i] < 0) return ORACLE_ERR_ARG;
        int pe = word[i] % o->npes;
        size_t off = table_off + 8 * (size_t)(word[i] / o->npes);
        uint64_t old;
        int rc = oracle_atomic(o, A_COMPARE_SWAP, 8, off, (uint64_t)value[i], (uint64_t)cond[i],
                               pe, &old);
        if (rc) return rc;
        if (fetched) fetched[i] = (int64_t)old;
    }
    return ORACLE_OK;
}

/* ---- collectives (Section 3.7.2) ------------------------------------------ */

/* A team is the PE set {start + i*stride, i = 0..size-1}. */
static int team_check(const oracle_t *o, int start, int stride, int size)
{
    if (size < 1 || stride < 1 || start < 0) return ORACLE_ERR_ARG;
    if (start + (size - 1) * stride >= o->npes) return ORACLE_ERR_INVALID_PE;
    return ORACLE_OK;
}

/* broadcast: every team member's dest receives the root's source ("Sync and
 * Broadcast").  `root` is an index inside the team.  root_writes_dest selects
 * whether the root's own dest is written too. */
int oracle_broadcastmem(oracle_t *o, int t_start, int t_stride, int t_size, size_t dest_off,
                        size_t src_off, size_t n, int root, int root_writes_dest)
{
    int rc = team_check(o, t_start, t_stride, t_size);
    if (rc) return rc;
    if (root < 0 || root >= t_size) return ORACLE_ERR_INVALID_PE;
    int root_pe = t_start + root * t_stride;
    rc = check(o, src_off, n, root_pe);
    if (rc) return rc;
    rc = check(o, dest_off, n, root_pe);
    if (rc) return rc;
    unsigned char *snap = (unsigned char *)malloc(n ? n : 1);
    if (!snap) return ORACLE_ERR_OOM;
    memcpy(snap, o->heap[root_pe] + src_off, n);
    for (int i = 0; i < t_size; ++i) {
        if (i == root && !root_writes_dest) continue;
        unsigned char *d = o->heap[t_start + i * t_stride] + dest_off;
        for (size_t k = 0; k < n; ++k) d[k] = snap[k];
    }
    free(snap);
    return ORACLE_OK;
}

/* fcollect: like an allgather with equal contributions -- block i of every
 * member's dest is the source of team member i. */
int oracle_fcollectmem(oracle_t *o, int t_start, int t_stride, int t_size, size_t dest_off,
                       size_t src_off, size_t n)
{
    int rc = team_check(o, t_start, t_stride, t_size);
    if (rc) return rc;
    rc = check(o, src_off, n, t_start);
    if (rc) return rc;
    if (n && (size_t)t_size > (o->heap_bytes - dest_off) / n) return ORACLE_ERR_NOT_SYMMETRIC;
    rc = check(o, dest_off, n * (size_t)t_size, t_start);
    if (rc) return rc;
    unsigned char *snap = (unsigned char *)malloc(n * (size_t)t_size + 1);
    if (!snap) return ORACLE_ERR_OOM;
    for (int i = 0; i < t_size; ++i)
        memcpy(snap + (size_t)i * n, o->heap[t_start + i * t_stride] + src_off, n);
    for (int q = 0; q < t_size; ++q) {
        unsigned char *d = o->heap[t_start + q * t_stride] + dest_off;
        for (size_t k = 0; k < n * (size_t)t_size; ++k) d[k] = snap[k];
    }
    free(snap);
    return ORACLE_OK;
}

/* collect: like fcollect with contributions of different sizes (Section 3.7.2 likens it to MPI's
 * allgather) -- every member's dest is the concatenation, in team order, of
 * the members' sources; member i contributes nbytes[i] bytes. */
int oracle_collectmem(oracle_t *o, int t_start, int t_stride, int t_size, size_t dest_off,
                      size_t src_off, const size_t *nbytes)
{
    int rc = team_check(o, t_start, t_stride, t_size);
    if (rc) return rc;
    size_t total = 0;
    for (int i = 0; i < t_size; ++i) {
        rc = check(o, src_off, nbytes[i], t_start + i * t_stride);
        if (rc) return rc;
        if (nbytes[i] > o->heap_bytes - total) return ORACLE_ERR_NOT_SYMMETRIC;
        total += nbytes[i];
    }
    rc = check(o, dest_off, total, t_start);
    if (rc) return rc;
    unsigned char *snap = (unsigned char *)malloc(total + 1);
    if (!snap) return ORACLE_ERR_OOM;
    size_t at = 0;
    for (int i = 0; i < t_size; ++i) {
        memcpy(snap + at, o->heap[t_start + i * t_stride] + src_off, nbytes[i]);
        at += nbytes[i];
    }
    for (int q = 0; q < t_size; ++q) {
        unsigned char *d = o->heap[t_start + q * t_stride] + dest_off;
        for (size_t k = 0; k < total; ++k) d[k] = snap[k];
    }
    free(snap);
    return ORACLE_OK;
}

/* alltoall (OpenSHMEM 1.5 team collective): block i of member q's dest is block q of member
 * i's source, blocks of n bytes: dest@q[i*n + k] = src@i[q*n + k]. */
int oracle_alltoallmem(oracle_t *o, int t_start, int t_stride, int t_size, size_t dest_off,
                       size_t src_off, size_t n)
{
    int rc = team_check(o, t_start, t_stride, t_size);
    if (rc) return rc;
    if (n && (size_t)t_size > o->heap_bytes / n) return ORACLE_ERR_NOT_SYMMETRIC;
    const size_t all = n * (size_t)t_size;
    rc = check(o, src_off, all, t_start);
    if (rc) return rc;
    rc = check(o, dest_off, all, t_start);
    if (rc) return rc;
    unsigned char *snap = (unsigned char *)malloc(all * (size_t)t_size + 1);
    if (!snap) return ORACLE_ERR_OOM;
    for (int i = 0; i < t_size; ++i)
        memcpy(snap + (size_t)i * all, o->heap[t_start + i * t_stride] + src_off, all);
    for (int q = 0; q < t_size; ++q) {
        unsigned char *d = o->heap[t_start + q * t_stride] + dest_off;
        for (int i = 0; i < t_size; ++i)
            for (size_t k = 0; k < n; ++k) d[(size_t)i * n + k] = snap[(size_t)i * all + (size_t)q * n + k];
    }
    free(snap);
    return ORACLE_OK;
}

/* One binary combine, `acc = acc op x`, in the element's own precision.
 * Integer sum and product wrap (computed unsigned); max/min keep the left
 * operand on ties: (x > acc) ? x : acc. */
#define COMBINE_INT(S, U)                                               \
    static S combine_##S(int op, S acc, S x)                            \
    {                                                                   \
        switch (op) {                                                   \
        case R_SUM: return (S)((U)acc + (U)x);                          \
        case R_PROD: return (S)((U)acc * (U)x);                         \
        case R_MAX: return (x > acc) ? x : acc;                         \
        case R_MIN: return (x < acc) ? x : acc;                         \
        case R_AND: return (S)((U)acc & (U)x);                          \
        case R_OR: return (S)((U)acc | (U)x);                           \
        default: return (S)((U)acc ^ (U)x);                             \
        }                                                               \
    }
COMBINE_INT(int32_t, uint32_t)
COMBINE_INT(int64_t, uint64_t)
COMBINE_INT(uint32_t, uint32_t)
COMBINE_INT(uint64_t, uint64_t)
/* 8- and 16-bit elements (integer types of 8 to 64 bits, Section 3.7.2): the unsigned type of the
 * same width keeps sum and product modulo 2^8 / 2^16 */
COMBINE_INT(int8_t, uint8_t)
COMBINE_INT(uint8_t, uint8_t)
COMBINE_INT(int16_t, uint16_t)
COMBINE_INT(uint16_t, uint16_t)

#define COMBINE_FP(F)                                                   \
    static F combine_##F(int op, F acc, F x)                            \
    {                                                                   \
        switch (op) {                                                   \
        case R_SUM: return acc + x;                                     \
        case R_PROD: return acc * x;                                    \
        case R_MAX: return (x > acc) ? x : acc;                         \
        default: return (x < acc) ? x : acc;                            \
        }                                                               \
    }
COMBINE_FP(float)
COMBINE_FP(double)

/* reduce: dest[j] on every member = ((s_0[j] op s_1[j]) op ...) op s_{P-1}[j],
 * a left fold in team order over a snapshot of all sources ("Reduction"). */
int oracle_reduce(oracle_t *o, int t_start, int t_stride, int t_size, size_t dest_off,
                  size_t src_off, size_t nreduce, int op, int dtype)
{
    int rc = team_check(o, t_start, t_stride, t_size);
    if (rc) return rc;
    size_t es = type_size(dtype);
    if (!es) return ORACLE_ERR_ARG;
    if (op < R_SUM || op > R_XOR) return ORACLE_ERR_ARG;
    if ((dtype == T_FLOAT || dtype == T_DOUBLE) && op > R_PROD) return ORACLE_ERR_ARG;
    if (dest_off % es || src_off % es) return ORACLE_ERR_ALIGN;
    if (nreduce > o->heap_bytes / es) return ORACLE_ERR_NOT_SYMMETRIC;
    rc = check(o, src_off, nreduce * es, t_start);
    if (rc) return rc;
    rc = check(o, dest_off, nreduce * es, t_start);
    if (rc) return rc;
    unsigned char *res = (unsigned char *)malloc(nreduce * es + 1);
    if (!res) return ORACLE_ERR_OOM;
    for (size_t j = 0; j < nreduce; ++j) {
#define FOLD(S)                                                                         \
        {                                                                               \
            S acc = ((const S *)(o->heap[t_start] + src_off))[j];                       \
            for (int i = 1; i < t_size; ++i)                                            \
                acc = combine_##S(op, acc,                                              \
                                  ((const S *)(o->heap[t_start + i * t_stride] + src_off))[j]); \
            ((S *)res)[j] = acc;                                                        \
        }
        switch (dtype) {
        case T_INT32: FOLD(int32_t) break;
        case T_INT64: FOLD(int64_t) break;
        case T_UINT32: FOLD(uint32_t) break;
        case T_UINT64: FOLD(uint64_t) break;
        case T_FLOAT: FOLD(float) break;
        case T_INT8: FOLD(int8_t) break;
        case T_UINT8: FOLD(uint8_t) break;
        case T_INT16: FOLD(int16_t) break;
        case T_UINT16: FOLD(uint16_t) break;
        default: FOLD(double) break;
        }
#undef FOLD
    }
    for (int q = 0; q < t_size; ++q)
        memcpy(o->heap[t_start + q * t_stride] + dest_off, res, nreduce * es);
    free(res);
    return ORACLE_OK;
}

/* ---- overlap workload: 5-point Jacobi --------------------------------------- */

/* One full-grid reference: `iters` sweeps of
 *   u'[i][j] = 0.25 * ((u[i-1][j] + u[i+1][j]) + (u[i][j-1] + u[i][j+1]))
 * on the interior of an ny x nx row-major grid; the outermost ring keeps its
 * input value (Dirichlet).  `u` is updated in place; `scratch` has the same
 * size.  *residual_sq = || u_iters - u_{iters-1} ||_2 squared over interior
 * cells, accumulated in row-major order (the caller takes the root). */
int oracle_jacobi(double *u, double *scratch, size_t ny, size_t nx, int iters, double *residual_sq)
{
    if (ny < 3 || nx < 3 || iters < 0) return ORACLE_ERR_ARG;
    double *a = u, *b = scratch;
    memcpy(b, a, ny * nx * sizeof(double));
    double res2 = 0.0;
    for (int it = 0; it < iters; ++it) {
        res2 = 0.0;
        for (size_t i = 1; i + 1 < ny; ++i)
            for (size_t j = 1; j + 1 < nx; ++j) {
                double ns = a[(i - 1) * nx + j] + a[(i + 1) * nx + j];
                double we = a[i * nx + j - 1] + a[i * nx + j + 1];
                double s = ns + we;
                double v = 0.25 * s;
                double d = v - a[i * nx + j];
                b[i * nx + j] = v;
                res2 += d * d;
            }
        double *t = a; a = b; b = t;
    }
    if (a != u) memcpy(u, a, ny * nx * sizeof(double));
    if (residual_sq) *residual_sq = res2;
    return ORACLE_OK;
}

/* The same computation written as the PE program: the grid's ny rows are cut
 * into npes row strips (the first ny mod npes strips get one extra row).  Each
 * PE keeps its strip plus one halo row above and below in two symmetric
 * buffers `buf_off[0]`, `buf_off[1]` of (max_rows + 2) * nx doubles; each sweep
 * every PE puts its first and last strip rows into its neighbours' halo rows
 * with put_signal (signal word = sweep number, one word per direction at
 * sig_off and sig_off + 8), checks the wait_until condition, then updates its
 * strip.  The caller scatters the initial grid with oracle_jacobi_scatter and
 * collects with oracle_jacobi_gather. */
static void strip_rows(size_t ny, int npes, int pe, size_t *first, size_t *rows)
{
    size_t base = ny / (size_t)npes, extra = ny % (size_t)npes;
    *rows = base + ((size_t)pe < extra ? 1 : 0);
    *first = (size_t)pe * base + ((size_t)pe < extra ? (size_t)pe : extra);
}

int oracle_jacobi_strip_rows(size_t ny, int npes, int pe, size_t *first, size_t *rows)
{
    if (npes < 1 || pe < 0 || pe >= npes) return ORACLE_ERR_INVALID_PE;
    strip_rows(ny, npes, pe, first, rows);
    return ORACLE_OK;
}

int oracle_jacobi_scatter(oracle_t *o, size_t buf_off, const double *grid, size_t ny, size_t nx)
{
    for (int p = 0; p < o->npes; ++p) {
        size_t first, rows;
        strip_rows(ny, o->npes, p, &first, &rows);
        int rc = check(o, buf_off, (rows + 2) * nx * 8, p);
        if (rc) return rc;
        double *b = (double *)(o->heap[p] + buf_off);
        /* strip row r sits at local row r + 1; halos are filled by the sweeps */
        memcpy(b + nx, grid + first * nx, rows * nx * 8);
    }
    return ORACLE_OK;
}

int oracle_jacobi_gather(const oracle_t *o, size_t buf_off, double *grid, size_t ny, size_t nx)
{
    for (int p = 0; p < o->npes; ++p) {
        size_t first, rows;
        strip_rows(ny, o->npes, p, &first, &rows);
        const double *b = (const double *)(o->heap[p] + buf_off);
        memcpy(grid + first * nx, b + nx, rows * nx * 8);
    }
    return ORACLE_OK;
}

int oracle_jacobi_strips(oracle_t *o, size_t buf0_off, size_t buf1_off, size_t sig_off, size_t ny,
                         size_t nx, int iters, double *residual_sq)
{
    if (ny < 3 || nx < 3 || iters < 0 || (size_t)o->npes > ny) return ORACLE_ERR_ARG;
    size_t off[2] = { buf0_off, buf1_off };
    int P = o->npes;
    double res2 = 0.0;
    /* both buffers start from the same strip contents, so that the Dirichlet
     * ring is present in whichever buffer a sweep writes */
    for (int p = 0; p < P; ++p) {
        size_t first, rows;
        strip_rows(ny, P, p, &first, &rows);
        int rc = check(o, off[1], (rows + 2) * nx * 8, p);
        if (rc) return rc;
        memcpy(o->heap[p] + off[1], o->heap[p] + off[0], (rows + 2) * nx * 8);
    }
    for (int it = 0; it < iters; ++it) {
        size_t cur = off[it & 1], nxt = off[(it + 1) & 1];
        uint64_t round = (uint64_t)it + 1;
        /* halo exchange by put_signal: my first row -> upper neighbour's bottom
         * halo, my last row -> lower neighbour's top halo */
        for (int p = 0; p < P; ++p) {
            size_t first, rows, nfirst, nrows;
            strip_rows(ny, P, p, &first, &rows);
            const double *mine = (const double *)(o->heap[p] + cur);
            if (p > 0) {
                strip_rows(ny, P, p - 1, &nfirst, &nrows);
                int rc = oracle_putmem_signal(o, p, cur + (nrows + 1) * nx * 8, mine + nx, nx * 8,
                                              sig_off + 8, round, SIG_SET, p - 1);
                if (rc) return rc;
            }
            if (p + 1 < P) {
                int rc = oracle_putmem_signal(o, p, cur, mine + rows * nx, nx * 8, sig_off, round,
                                              SIG_SET, p + 1);
                if (rc) return rc;
            }
        }
        res2 = 0.0;
        for (int p = 0; p < P; ++p) {
            size_t first, rows;
            strip_rows(ny, P, p, &first, &rows);
            if (p > 0 && oracle_test(o, p, sig_off, C_GE, round) != 1) return ORACLE_ERR_ARG;
            if (p + 1 < P && oracle_test(o, p, sig_off + 8, C_GE, round) != 1) return ORACLE_ERR_ARG;
            const double *a = (const double *)(o->heap[p] + cur);
            double *b = (double *)(o->heap[p] + nxt);
            for (size_t r = 1; r <= rows; ++r) {
                size_t gi = first + r - 1; /* global row */
                if (gi == 0 || gi == ny - 1) continue; /* Dirichlet rows */
                for (size_t j = 1; j + 1 < nx; ++j) {
                    double ns = a[(r - 1) * nx + j] + a[(r + 1) * nx + j];
                    double we = a[r * nx + j - 1] + a[r * nx + j + 1];
                    double s = ns + we;
                    double v = 0.25 * s;
                    double d = v - a[r * nx + j];
                    b[r * nx + j] = v;
                    res2 += d * d;
                }
            }
        }
    }
    if (residual_sq) *residual_sq = res2;
    return ORACLE_OK;
}

/* Exact value of one cell after `iters` sweeps, computed from its dependency
 * cone only.  `win` is the h x w window of the INITIAL grid whose top-left cell
 * is global (i0, j0); it must reach `iters` cells from (ci, cj) in every
 * direction or stop at the grid's edge.  The window is swept `iters` times;
 * window-edge cells that are not grid-edge cells are left stale, which after k
 * sweeps has corrupted only cells within distance k-1 of the window edge and so
 * never reaches the centre. */
int oracle_jacobi_cell(const double *win, size_t h, size_t w, size_t i0, size_t j0, size_t ny,
                       size_t nx, int iters, size_t ci, size_t cj, double *value_out)
{
    if (iters < 0 || ci < i0 || cj < j0 || ci >= i0 + h || cj >= j0 + w) return ORACLE_ERR_ARG;
    if (i0 + h > ny || j0 + w > nx) return ORACLE_ERR_ARG;
    size_t r = (size_t)iters;
    /* the window must contain the cone */
    if ((ci - i0 < r && i0 != 0) || (i0 + h - 1 - ci < r && i0 + h != ny)) return ORACLE_ERR_ARG;
    if ((cj - j0 < r && j0 != 0) || (j0 + w - 1 - cj < r && j0 + w != nx)) return ORACLE_ERR_ARG;
    double *a = (double *)malloc(h * w * 8), *b = (double *)malloc(h * w * 8);
    if (!a || !b) { free(a); free(b); return ORACLE_ERR_OOM; }
    memcpy(a, win, h * w * 8);
    memcpy(b, win, h * w * 8);
    for (int it = 0; it < iters; ++it) {
        for (size_t i = 0; i < h; ++i)
            for (size_t j = 0; j < w; ++j) {
                size_t gi = i0 + i, gj = j0 + j;
                if (gi == 0 || gj == 0 || gi == ny - 1 || gj == nx - 1) continue; /* Dirichlet */
                if (i == 0 || j == 0 || i == h - 1 || j == w - 1) {
                    b[i * w + j] = a[i * w + j]; /* outside the cone: stale */
                    continue;
                }
                double ns = a[(i - 1) * w + j] + a[(i + 1) * w + j];
                double we = a[i * w + j - 1] + a[i * w + j + 1];
                double s = ns + we;
                b[i * w + j] = 0.25 * s;
            }
        double *t = a; a = b; b = t;
    }
    *value_out = a[(ci - i0) * w + (cj - j0)];
    free(a); free(b);
    return ORACLE_OK;
}
