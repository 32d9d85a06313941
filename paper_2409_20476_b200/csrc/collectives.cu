/* Team synchronisation and collectives (Section 3.7.2 of the paper): push sync, push
 * broadcast / fcollect, reduce in its duplicated and split-by-address forms.
 *
 * Host-called collectives run as ONE launch for the whole team on the team stream; the
 * launch boundary is their synchronisation.  The device-resident forms (one work-group
 * per PE with in-kernel push sync) are exercised by ishmemx_collective_on_device, a
 * co-resident (cooperative) launch. */
#include "internal.h"

struct coll_args {
    ishmem_team_t team;
    char *dest;       /* PE 0's copy (symmetric address) */
    const char *src;
    size_t n;         /* bytes (broadcast, fcollect) or elements (reduce) */
    int root;
    int groups;       /* blocks per member */
    int duplicated;   /* reduce: every member folds everything into its own dest */
    int repeat;
    unsigned staging_bytes; /* dynamic shared memory for the TMA push ring (0: loads/stores) */
    unsigned tile_vpt;      /* reduce: 16-byte vectors per thread in one tile */
    unsigned push_tile;     /* broadcast / fcollect by loads and stores: bytes per tile */
};

/* local address on `ctx`'s PE of a symmetric address given as PE 0's copy */
__device__ __forceinline__ char *local_of(const ishmem_ctx_t *ctxs, const ishmem_ctx_t *ctx, const char *sym0)
{
    return (char *)sym0 + (ctx->heap_base - ctxs[0].heap_base);
}

/* vector-slot range [lo, hi) of part `k` of `parts` over `n` slots */
__device__ __forceinline__ void part_of(size_t n, unsigned k, unsigned parts, size_t *lo, size_t *hi)
{
    *lo = (size_t)(((unsigned __int128)n * k) / parts);
    *hi = (size_t)(((unsigned __int128)n * (k + 1)) / parts);
}

/* ---- broadcast: the root's blocks push slices of the source to every member ------------- */
__global__ void __launch_bounds__(1024) k_broadcast(const ishmem_ctx_t *ctxs, coll_args a)
{
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ long long delta[ISHMEM_MAX_PES];
    const ishmemi_team t = ctxs[0].teams[a.team];
    const ishmem_ctx_t *ctx = ctxs + (t.start + a.root * t.stride);
    if (!ishmemi::team_deltas(ctx, t, delta)) return;
    /* the root's blocks take chunks of the message round-robin */
    ishmemx_staging_t st = {a.staging_bytes ? dyn_smem : nullptr, a.staging_bytes};
    ishmemi::wg_push(ctx, local_of(ctxs, ctx, a.dest), delta, t.size, ctx->bcast_root_dest ? -1 : a.root,
                     local_of(ctxs, ctx, a.src), a.n, st, blockIdx.x, gridDim.x, a.push_tile);
}

/* ---- fcollect: member i's blocks push slices of its source into block i of every dest ---- */
__global__ void __launch_bounds__(1024) k_fcollect(const ishmem_ctx_t *ctxs, coll_args a)
{
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ long long delta[ISHMEM_MAX_PES];
    const ishmemi_team t = ctxs[0].teams[a.team];
    const unsigned me = blockIdx.x % (unsigned)t.size, g = blockIdx.x / (unsigned)t.size;
    const ishmem_ctx_t *ctx = ctxs + (t.start + (int)me * t.stride);
    if (!ishmemi::team_deltas(ctx, t, delta)) return;
    ishmemx_staging_t st = {a.staging_bytes ? dyn_smem : nullptr, a.staging_bytes};
    ishmemi::wg_push(ctx, local_of(ctxs, ctx, a.dest) + (size_t)me * a.n, delta, t.size, -1,
                     local_of(ctxs, ctx, a.src), a.n, st, g, (size_t)a.groups, a.push_tile);
}

/* ---- broadcast / fcollect of large messages as (tile, source member, destination) triples --------
 * One block copies one 32 KiB tile of one member's source into one member's destination, like a tile
 * of a put; the destination runs fastest, then the source member, then the tile, so the P blocks that
 * read the same source tile start together (one of them brings it from DRAM, the others find it in
 * L2) and the running blocks sweep one window of every source and destination in launch order.  The
 * fan-out kernels above store each loaded vector P times from the same thread, which wins on large
 * teams; on small teams the P separate copies move more bytes per second (single launches, broadcast of
 * 256 MiB / fcollect of 64 MiB per PE, fan-out against triples: 4 PEs 5.1 / 4.9 against 6.2 / 6.1 TB/s,
 * 8 PEs 6.2 / 6.0 against 6.0 / 6.0, 12 PEs 6.4 / 6.4 against 5.9 / 5.8).  members = 1: broadcast from
 * `root`; members = team size: fcollect. */
#define PUSH_PAIR_TILE 32768u
__global__ void __launch_bounds__(256) k_push_pairs(const ishmem_ctx_t *ctxs, coll_args a, int members, int skip)
{
    const ishmemi_team t = ctxs[0].teams[a.team];
    const size_t P = (size_t)t.size, per = (a.n + PUSH_PAIR_TILE - 1) / PUSH_PAIR_TILE;
    const size_t total = per * (size_t)members * P;
    for (size_t b = blockIdx.x; b < total; b += gridDim.x) {
        const int q = (int)(b % P), i = (int)((b / P) % (size_t)members);
        const size_t o = (b / (P * (size_t)members)) * PUSH_PAIR_TILE;
        if (q == skip) continue;
        const int from = members == 1 ? a.root : i;
        const ishmem_ctx_t *ctx = ctxs + (t.start + from * t.stride);
        /* the pushing PE names the destination by its own copy and translates it to member q */
        char *d = ishmemi::translate(ctx, local_of(ctxs, ctx, a.dest), t.start + q * t.stride);
        if (!d) return;
        const size_t len = a.n - o < PUSH_PAIR_TILE ? a.n - o : PUSH_PAIR_TILE;
        ishmemi::copy_bytes(d + (members == 1 ? 0 : (size_t)i * a.n) + o, local_of(ctxs, ctx, a.src) + o, len, threadIdx.x,
                            blockDim.x);
    }
}
/* ISHMEMX_OPT_PUSH_SHAPE: 1 = fan-out tiles, 2 = (tile, member, destination) triples, 0 = by measurement:
 * triples for messages of at least 4 MiB on teams of up to 6 members */
static bool push_as_pairs(size_t nbytes, int team_size)
{
    const long long shape = g_ishmem.opt[ISHMEMX_OPT_PUSH_SHAPE];
    if (shape == 1) return false;
    if (shape == 2) return true;
    return g_ishmem.coll_groups == 0 && nbytes >= ((size_t)4 << 20) && team_size <= 6;
}
static int launch_push_pairs(cudaStream_t s, const coll_args &a, int members, int P, int skip)
{
    const size_t per = (a.n + PUSH_PAIR_TILE - 1) / PUSH_PAIR_TILE, total = per * (size_t)members * (size_t)P;
    k_push_pairs<<<(unsigned)(total < 0x7fffffffu ? total : 0x7fffffffu), 256, 0, s>>>(g_ishmem.d_ctx, a, members, skip);
    ishmemi_count_launch();
    return ishmemi_check_launch("k_push_pairs");
}

/* ---- collect: fcollect with a size and an offset per member ------------------------------------ */
struct collect_args {
    ishmem_team_t team;
    char *dest;
    const char *src;
    int groups;
    unsigned tile;
    unsigned long long nbytes[ISHMEM_MAX_PES], offset[ISHMEM_MAX_PES];
};
__global__ void __launch_bounds__(1024) k_collect(const ishmem_ctx_t *ctxs, collect_args a)
{
    __shared__ long long delta[ISHMEM_MAX_PES];
    const ishmemi_team t = ctxs[0].teams[a.team];
    const unsigned me = blockIdx.x % (unsigned)t.size, g = blockIdx.x / (unsigned)t.size;
    const ishmem_ctx_t *ctx = ctxs + (t.start + (int)me * t.stride);
    if (!ishmemi::team_deltas(ctx, t, delta)) return;
    ishmemx_staging_t st = {nullptr, 0};
    ishmemi::wg_push(ctx, local_of(ctxs, ctx, a.dest) + a.offset[me], delta, t.size, -1, local_of(ctxs, ctx, a.src),
                     (size_t)a.nbytes[me], st, g, (size_t)a.groups, a.tile);
}

/* ---- alltoall: member i's blocks store block q of its source into block i of member q's dest ---- */
__global__ void __launch_bounds__(1024) k_alltoall(const ishmem_ctx_t *ctxs, coll_args a)
{
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ long long delta[ISHMEM_MAX_PES];
    const ishmemi_team t = ctxs[0].teams[a.team];
    const unsigned me = blockIdx.x % (unsigned)t.size, g = blockIdx.x / (unsigned)t.size;
    const ishmem_ctx_t *ctx = ctxs + (t.start + (int)me * t.stride);
    if (!ishmemi::team_deltas(ctx, t, delta)) return;
    const char *src = local_of(ctxs, ctx, a.src);
    char *dest = local_of(ctxs, ctx, a.dest) + (size_t)me * a.n;
    /* (destination, tile) pairs dealt round-robin, the destination running fastest so that
     * consecutive tiles go to different PEs */
    const size_t tile = a.push_tile, per = (a.n + tile - 1) / tile, total = per * (size_t)t.size;
    for (size_t k = g; k < total; k += (size_t)a.groups) {
        const size_t q = k % (size_t)t.size, o = (k / (size_t)t.size) * tile;
        const size_t len = a.n - o < tile ? a.n - o : tile;
        if (a.staging_bytes) {
            /* large blocks: every tile streams through the TMA ring of this block */
            ishmemx_staging_t st = {dyn_smem, a.staging_bytes};
            if (ishmemi::wg_copy(ctx, dest + delta[q] + o, src + q * a.n + o, len, st, true)) return;
            __syncthreads(); /* the ring's shared memory is reused by the next tile */
        } else {
            ishmemi::copy_bytes(dest + delta[q] + o, src + q * a.n + o, len, threadIdx.x, blockDim.x);
        }
    }
}

/* ---- reduce ------------------------------------------------------------------------------- */
/* split: member q owns a contiguous address range, folds it from all sources in team order
 * and stores the result into every member's dest (traffic: each source and each dest once).
 * duplicated: member q folds the whole range and stores into its own dest only. */
template <typename T, int OP>
__global__ void __launch_bounds__(512, 2) k_reduce(const ishmem_ctx_t *ctxs, coll_args a)
{
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ long long delta[ISHMEM_MAX_PES];
    const ishmemi_team t = ctxs[0].teams[a.team];
    const unsigned me = blockIdx.x % (unsigned)t.size, g = blockIdx.x / (unsigned)t.size;
    const ishmem_ctx_t *ctx = ctxs + (t.start + (int)me * t.stride);
    if (!ishmemi::team_deltas(ctx, t, delta)) return;
    constexpr size_t EPV = 16 / sizeof(T);
    const char *src = local_of(ctxs, ctx, a.src);
    char *dest = local_of(ctxs, ctx, a.dest);
    const int dst0 = a.duplicated ? (int)me : 0, ndst = a.duplicated ? 1 : t.size;
    const unsigned tid = threadIdx.x, nthr = blockDim.x;
    if ((((uintptr_t)src | (uintptr_t)dest) & 15u) != 0) {
        /* buffers aligned to the element only: contiguous element ranges, element by element */
        size_t lo = 0, hi = a.n, glo, ghi;
        if (!a.duplicated) part_of(a.n, me, (unsigned)t.size, &lo, &hi);
        part_of(hi - lo, g, (unsigned)a.groups, &glo, &ghi);
        ishmemi::fold_range<T, OP, 1, 4>(src, dest, delta, t.size, dst0, ndst, lo + glo, lo + ghi, tid, nthr);
        return;
    }
    /* The address range is cut into tiles that the blocks take round-robin, so that at any
     * moment the running blocks cover one contiguous window of every source and destination
     * (whole DRAM rows, all channels).  Split form: tile k belongs to member k mod P -- still
     * a split of the work by address across PEs; duplicated form: each member's blocks sweep
     * all tiles. */
    const size_t nv = a.n / EPV;
    const size_t tile = (size_t)nthr * a.tile_vpt;
    const size_t ntiles = (nv + tile - 1) / tile;
    const size_t first = a.duplicated ? g : blockIdx.x, stride = a.duplicated ? (size_t)a.groups : gridDim.x;
    if (a.staging_bytes) {
        ishmemx_staging_t st = {dyn_smem, a.staging_bytes};
        ishmemi::bulk_fold_ring<T, OP>(ctx, src, dest, delta, t.size, dst0, ndst, nv * 16, st, first, stride);
    } else {
        for (size_t k = first; k < ntiles; k += stride) {
            const size_t v0 = k * tile, v1 = (v0 + tile < nv) ? v0 + tile : nv;
            ishmemi::fold_vectors<T, OP, 1, 4>(src, dest, delta, t.size, dst0, ndst, v0, v1, tid, nthr);
        }
    }
    /* elements past the last whole vector */
    if (first == 0)
        ishmemi::fold_range<T, OP, 1, 4>(src, dest, delta, t.size, dst0, ndst, nv * EPV, a.n, tid, nthr);
}

typedef void (*reduce_kernel_t)(const ishmem_ctx_t *, coll_args);

template <typename T>
static reduce_kernel_t pick_arith(int op)
{
    switch (op) {
    case ISHMEM_OP_SUM: return k_reduce<T, ISHMEM_OP_SUM>;
    case ISHMEM_OP_MAX: return k_reduce<T, ISHMEM_OP_MAX>;
    case ISHMEM_OP_MIN: return k_reduce<T, ISHMEM_OP_MIN>;
    case ISHMEM_OP_PROD: return k_reduce<T, ISHMEM_OP_PROD>;
    default: return nullptr;
    }
}
template <typename T>
static reduce_kernel_t pick_int(int op)
{
    switch (op) {
    case ISHMEM_OP_AND: return k_reduce<T, ISHMEM_OP_AND>;
    case ISHMEM_OP_OR: return k_reduce<T, ISHMEM_OP_OR>;
    case ISHMEM_OP_XOR: return k_reduce<T, ISHMEM_OP_XOR>;
    default: return pick_arith<T>(op);
    }
}
static reduce_kernel_t pick_reduce(int op, int dtype)
{
    switch (dtype) {
    case ISHMEM_T_INT32: return pick_int<int>(op);
    case ISHMEM_T_INT64: return pick_int<long long>(op);
    case ISHMEM_T_UINT32: return pick_int<unsigned>(op);
    case ISHMEM_T_UINT64: return pick_int<unsigned long long>(op);
    case ISHMEM_T_FLOAT: return pick_arith<float>(op);
    case ISHMEM_T_DOUBLE: return pick_arith<double>(op);
    case ISHMEM_T_INT8: return pick_int<signed char>(op);
    case ISHMEM_T_UINT8: return pick_int<unsigned char>(op);
    case ISHMEM_T_INT16: return pick_int<short>(op);
    case ISHMEM_T_UINT16: return pick_int<unsigned short>(op);
    default: return nullptr;
    }
}
static size_t dtype_size(int dtype)
{
    switch (dtype) {
    case ISHMEM_T_INT32: case ISHMEM_T_UINT32: case ISHMEM_T_FLOAT: return 4;
    case ISHMEM_T_INT64: case ISHMEM_T_UINT64: case ISHMEM_T_DOUBLE: return 8;
    case ISHMEM_T_INT8: case ISHMEM_T_UINT8: return 1;
    case ISHMEM_T_INT16: case ISHMEM_T_UINT16: return 2;
    default: return 0;
    }
}

/* ---- device-resident forms: one work-group per member, in-kernel push sync ---------------- */
/* WHICH: 0 broadcast, 1 fcollect, 2 reduce<T, OP>, 3 sync, 4 alltoall, 5 collect (member i of the
 * team contributes n * ((i mod 3) + 1) / 3 bytes: a fixed ragged pattern for tests) */
template <int WHICH, typename T, int OP>
__global__ void __launch_bounds__(1024) k_collective_on_device(const ishmem_ctx_t *ctxs, coll_args a)
{
    const ishmemi_team t = ctxs[0].teams[a.team];
    /* the context in shared memory: the collectives below look PEs up many times, each after the
     * acquire that ends a sync */
    __shared__ ishmem_ctx_t ctx_copy;
    const ishmem_ctx_t *ctx = ctxs + (t.start + (int)blockIdx.x * t.stride);
    char *d = a.dest ? local_of(ctxs, ctx, a.dest) : nullptr;
    const char *s = a.src ? local_of(ctxs, ctx, a.src) : nullptr;
    ctx = ishmemx_ctx_stage_work_group(&ctx_copy, ctx);
    for (int r = 0; r < a.repeat; ++r) {
        int rc;
        if (WHICH == 0) rc = ishmemx_broadcastmem_work_group(ctx, a.team, d, s, a.n, a.root);
        else if (WHICH == 1) rc = ishmemx_fcollectmem_work_group(ctx, a.team, d, s, a.n);
        else if (WHICH == 2) rc = ishmemx_reduce_work_group<T, OP>(ctx, a.team, (T *)d, (const T *)s, a.n);
        else if (WHICH == 4) rc = ishmemx_alltoallmem_work_group(ctx, a.team, d, s, a.n);
        else if (WHICH == 5) rc = ishmemx_collectmem_work_group(ctx, a.team, d, s, a.n * (size_t)(blockIdx.x % 3 + 1) / 3);
        else rc = ishmemx_team_sync_work_group(ctx, a.team);
        if (rc) return; /* the error is latched; every member gives up the same way */
    }
}

template <typename T>
static reduce_kernel_t pick_dev_arith(int op)
{
    switch (op) {
    case ISHMEM_OP_SUM: return k_collective_on_device<2, T, ISHMEM_OP_SUM>;
    case ISHMEM_OP_MAX: return k_collective_on_device<2, T, ISHMEM_OP_MAX>;
    case ISHMEM_OP_MIN: return k_collective_on_device<2, T, ISHMEM_OP_MIN>;
    case ISHMEM_OP_PROD: return k_collective_on_device<2, T, ISHMEM_OP_PROD>;
    default: return nullptr;
    }
}
template <typename T>
static reduce_kernel_t pick_dev_int(int op)
{
    switch (op) {
    case ISHMEM_OP_AND: return k_collective_on_device<2, T, ISHMEM_OP_AND>;
    case ISHMEM_OP_OR: return k_collective_on_device<2, T, ISHMEM_OP_OR>;
    case ISHMEM_OP_XOR: return k_collective_on_device<2, T, ISHMEM_OP_XOR>;
    default: return pick_dev_arith<T>(op);
    }
}
static reduce_kernel_t pick_dev(int which, int op, int dtype)
{
    if (which == 0) return k_collective_on_device<0, int, 0>;
    if (which == 1) return k_collective_on_device<1, int, 0>;
    if (which == 3) return k_collective_on_device<3, int, 0>;
    if (which == 4) return k_collective_on_device<4, int, 0>;
    if (which == 5) return k_collective_on_device<5, int, 0>;
    switch (dtype) {
    case ISHMEM_T_INT32: return pick_dev_int<int>(op);
    case ISHMEM_T_INT64: return pick_dev_int<long long>(op);
    case ISHMEM_T_UINT32: return pick_dev_int<unsigned>(op);
    case ISHMEM_T_UINT64: return pick_dev_int<unsigned long long>(op);
    case ISHMEM_T_FLOAT: return pick_dev_arith<float>(op);
    case ISHMEM_T_DOUBLE: return pick_dev_arith<double>(op);
    case ISHMEM_T_INT8: return pick_dev_int<signed char>(op);
    case ISHMEM_T_UINT8: return pick_dev_int<unsigned char>(op);
    case ISHMEM_T_INT16: return pick_dev_int<short>(op);
    case ISHMEM_T_UINT16: return pick_dev_int<unsigned short>(op);
    default: return nullptr;
    }
}

/* ---- host side ---------------------------------------------------------------------------- */

static int team_of(ishmem_team_t team, ishmemi_team *out)
{
    auto &g = g_ishmem;
    if (team < 0 || team >= ISHMEM_MAX_TEAMS || !g.teams[team].valid) return ISHMEM_ERR_ARG;
    *out = g.teams[team];
    return ISHMEM_OK;
}

/* Launch shape of a push collective (broadcast: 1 pushing member; fcollect: `members`), each
 * pushing `bytes` to `ndst` destinations by loads and stores: one tile per block.  Blocks start in
 * index order, so at any moment the running blocks cover one short contiguous window of the source
 * and of every destination; on this GPU that order moves more bytes per second than a resident
 * grid whose blocks each stream a long range of their own, by loads and stores or by the TMA ring
 * (broadcast of 256 MiB to 12 PEs: 6.5 against 5.6 TB/s).  The tile is 8 KiB -- one 16-byte vector
 * per thread of a 512-thread block, stored to every destination -- and shrinks down to 2 KiB so
 * that a medium message still reaches every SM twice. */
struct push_shape {
    int blocks_per_member, threads;
    unsigned staging, tile;
};
static push_shape push_geometry(size_t bytes, int members, int ndst)
{
    auto &g = g_ishmem;
    push_shape sh = {1, g.coll_threads, 0, 16384};
    if (g.coll_groups > 0) { /* caller-shaped */
        sh.blocks_per_member = g.coll_groups;
        return sh;
    }
    const size_t aim = ((size_t)g.sm_count * 2 + members - 1) / members;
    size_t tile = (bytes / aim + 2047) & ~(size_t)2047;
    if (tile < 2048) tile = 2048;
    if (tile > 8192) tile = 8192;
    if (sh.threads > 512) sh.threads = 512;
    size_t want = (bytes + tile - 1) / tile;
    const size_t most = (size_t)0x7fffffff / (size_t)members; /* grid limit */
    sh.tile = (unsigned)tile;
    sh.blocks_per_member = (int)(want < 1 ? 1 : (want < most ? want : most));
    if (bytes <= 4096 * (size_t)ndst && sh.threads > 256) sh.threads = 256;
    return sh;
}

static int launch_sync_kernel(ishmem_team_t team, int repeat)
{
    auto &g = g_ishmem;
    ishmemi_team t;
    int rc = team_of(team, &t);
    if (rc) return rc;
    cudaStream_t s;
    if ((rc = ishmemi_team_stream_begin(team, &s))) return rc;
    coll_args a = {};
    a.team = team;
    a.repeat = repeat;
    const ishmem_ctx_t *ctxs = g.d_ctx;
    void *params[] = {(void *)&ctxs, (void *)&a};
    rc = ishmemi_cuda(cudaLaunchCooperativeKernel((void *)pick_dev(3, 0, 0), dim3(t.size), dim3(64),
                                                  params, 0, s),
                      "cudaLaunchCooperativeKernel(sync)");
    ishmemi_count_launch();
    ishmemi_team_stream_end();
    return rc;
}

extern "C" int ishmem_team_sync(ishmem_team_t team)
{
    ISHMEMI_REQUIRE_INIT();
    return launch_sync_kernel(team, 1);
}
extern "C" int ishmem_sync_all(void)
{
    ISHMEMI_REQUIRE_INIT();
    return launch_sync_kernel(ISHMEM_TEAM_WORLD, 1);
}
extern "C" int ishmem_barrier_all(void)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    int rc;
    for (int p = 0; p < g.npes; ++p)
        if ((rc = ishmem_quiet(p))) return rc;
    if ((rc = launch_sync_kernel(ISHMEM_TEAM_WORLD, 1))) return rc;
    ISHMEMI_CUDA(cudaStreamSynchronize(g.team_stream));
    return ISHMEM_OK;
}

static int check_sym2(const void *dest, size_t dbytes, const void *src, size_t sbytes)
{
    if (ishmemi_sym_offset(dest, dbytes) < 0 || ishmemi_sym_offset(src, sbytes) < 0)
        return ISHMEM_ERR_NOT_SYMMETRIC;
    return ISHMEM_OK;
}

extern "C" int ishmem_broadcastmem(ishmem_team_t team, void *dest, const void *src, size_t nbytes, int root)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    ishmemi_team t;
    int rc = team_of(team, &t);
    if (rc) return rc;
    if (root < 0 || root >= t.size) return ISHMEM_ERR_INVALID_PE;
    if ((rc = check_sym2(dest, nbytes, src, nbytes))) return rc;
    cudaStream_t s;
    if ((rc = ishmemi_team_stream_begin(team, &s))) return rc;
    if (nbytes == 0) {
        ishmemi_team_stream_end();
        return ISHMEM_OK;
    }
    if (nbytes >= g.cutover[1]) {
        /* copy engine: one transfer per destination */
        size_t doff = (size_t)ishmemi_sym_offset(dest, nbytes), soff = (size_t)ishmemi_sym_offset(src, nbytes);
        int root_pe = t.start + root * t.stride;
        for (int i = 0; i < t.size && !rc; ++i) {
            if (i == root && !g.bcast_root_dest) continue;
            int q = t.start + i * t.stride;
            rc = ishmemi_cuda(cudaMemcpyAsync(g.base + (size_t)q * g.heap_bytes + doff,
                                              g.base + (size_t)root_pe * g.heap_bytes + soff, nbytes,
                                              cudaMemcpyDeviceToDevice, s),
                              "cudaMemcpyAsync(broadcast)");
        }
    } else {
        coll_args a = {};
        a.team = team;
        a.dest = (char *)dest;
        a.src = (const char *)src;
        a.n = nbytes;
        a.root = root;
        if (push_as_pairs(nbytes, t.size)) {
            rc = launch_push_pairs(s, a, 1, t.size, g.bcast_root_dest ? -1 : root);
        } else {
            const push_shape sh = push_geometry(nbytes, 1, t.size);
            a.staging_bytes = sh.staging;
            a.push_tile = sh.tile;
            k_broadcast<<<sh.blocks_per_member, sh.threads, sh.staging, s>>>(g.d_ctx, a);
            ishmemi_count_launch();
            rc = ishmemi_check_launch("k_broadcast");
        }
    }
    ishmemi_team_stream_end();
    return rc;
}

extern "C" int ishmem_fcollectmem(ishmem_team_t team, void *dest, const void *src, size_t nbytes)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    ishmemi_team t;
    int rc = team_of(team, &t);
    if (rc) return rc;
    if (nbytes && (size_t)t.size > (size_t)-1 / nbytes) return ISHMEM_ERR_ARG;
    if ((rc = check_sym2(dest, nbytes * t.size, src, nbytes))) return rc;
    cudaStream_t s;
    if ((rc = ishmemi_team_stream_begin(team, &s))) return rc;
    if (nbytes == 0) {
        ishmemi_team_stream_end();
        return ISHMEM_OK;
    }
    if (nbytes >= g.cutover[2]) {
        size_t doff = (size_t)ishmemi_sym_offset(dest, nbytes), soff = (size_t)ishmemi_sym_offset(src, nbytes);
        for (int i = 0; i < t.size && !rc; ++i)
            for (int j = 0; j < t.size && !rc; ++j) {
                int from = t.start + i * t.stride, to = t.start + j * t.stride;
                rc = ishmemi_cuda(cudaMemcpyAsync(g.base + (size_t)to * g.heap_bytes + doff + (size_t)i * nbytes,
                                                  g.base + (size_t)from * g.heap_bytes + soff, nbytes,
                                                  cudaMemcpyDeviceToDevice, s),
                                  "cudaMemcpyAsync(fcollect)");
            }
    } else {
        coll_args a = {};
        a.team = team;
        a.dest = (char *)dest;
        a.src = (const char *)src;
        a.n = nbytes;
        if (push_as_pairs(nbytes, t.size)) {
            rc = launch_push_pairs(s, a, t.size, t.size, -1);
        } else {
            const push_shape sh = push_geometry(nbytes, t.size, t.size);
            a.groups = sh.blocks_per_member;
            a.staging_bytes = sh.staging;
            a.push_tile = sh.tile;
            k_fcollect<<<a.groups * t.size, sh.threads, sh.staging, s>>>(g.d_ctx, a);
            ishmemi_count_launch();
            rc = ishmemi_check_launch("k_fcollect");
        }
    }
    ishmemi_team_stream_end();
    return rc;
}

extern "C" int ishmem_collectmem(ishmem_team_t team, void *dest, const void *src, const size_t *nbytes_per_member)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    ishmemi_team t;
    int rc = team_of(team, &t);
    if (rc) return rc;
    if (!nbytes_per_member) return ISHMEM_ERR_ARG;
    collect_args a = {};
    size_t total = 0, largest = 0;
    for (int i = 0; i < t.size; ++i) {
        const size_t n = nbytes_per_member[i];
        if (n > g.heap_bytes || total > g.heap_bytes - n) return ISHMEM_ERR_NOT_SYMMETRIC;
        a.nbytes[i] = n;
        a.offset[i] = total;
        total += n;
        if (n > largest) largest = n;
    }
    if ((rc = check_sym2(dest, total, src, largest))) return rc;
    const char *d = (const char *)dest, *sp = (const char *)src;
    if (total && d < sp + largest && sp < d + total) return ISHMEM_ERR_ARG;
    cudaStream_t s;
    if ((rc = ishmemi_team_stream_begin(team, &s))) return rc;
    if (total) {
        a.team = team;
        a.dest = (char *)dest;
        a.src = sp;
        const push_shape sh = push_geometry(largest, t.size, t.size); /* sized for the largest contribution */
        a.groups = sh.blocks_per_member;
        a.tile = sh.tile;
        k_collect<<<a.groups * t.size, sh.threads, 0, s>>>(g.d_ctx, a);
        ishmemi_count_launch();
        rc = ishmemi_check_launch("k_collect");
    }
    ishmemi_team_stream_end();
    return rc;
}

extern "C" int ishmem_alltoallmem(ishmem_team_t team, void *dest, const void *src, size_t nbytes)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    ishmemi_team t;
    int rc = team_of(team, &t);
    if (rc) return rc;
    if (nbytes && (size_t)t.size > (size_t)-1 / nbytes) return ISHMEM_ERR_ARG;
    const size_t all = nbytes * t.size;
    if ((rc = check_sym2(dest, all, src, all))) return rc;
    const char *d = (const char *)dest, *sp = (const char *)src;
    if (all && d < sp + all && sp < d + all) return ISHMEM_ERR_ARG;
    cudaStream_t s;
    if ((rc = ishmemi_team_stream_begin(team, &s))) return rc;
    if (nbytes) {
        coll_args a = {};
        a.team = team;
        a.dest = (char *)dest;
        a.src = sp;
        a.n = nbytes;
        /* one (destination, tile) pair per block, the tile shrinking from 32 to 2 KiB while the
         * grid would not fill every SM four times */
        size_t tile = 32768;
        const size_t aim = ((size_t)g.sm_count * 4 + t.size - 1) / t.size;
        while (tile > 2048 && (all + tile - 1) / tile < aim) tile >>= 1;
        size_t want = ((nbytes + tile - 1) / tile) * t.size;
        const size_t most = (size_t)0x7fffffff / (size_t)t.size;
        a.push_tile = (unsigned)tile;
        a.groups = g.coll_groups > 0 ? g.coll_groups : (int)(want < 1 ? 1 : (want < most ? want : most));
        const int threads = (all <= 65536 || g.coll_groups == 0) ? 256 : g.coll_threads;
        k_alltoall<<<a.groups * t.size, threads, a.staging_bytes, s>>>(g.d_ctx, a);
        ishmemi_count_launch();
        rc = ishmemi_check_launch("k_alltoall");
    }
    ishmemi_team_stream_end();
    return rc;
}

template <typename T>
static int typed_collect(ishmem_team_t team, T *dest, const T *src, const size_t *nelems)
{
    ISHMEMI_REQUIRE_INIT();
    ishmemi_team t;
    int rc = team_of(team, &t);
    if (rc) return rc;
    if (!nelems) return ISHMEM_ERR_ARG;
    if (((uintptr_t)dest | (uintptr_t)src) % sizeof(T)) return ISHMEM_ERR_ALIGN;
    size_t bytes[ISHMEM_MAX_PES];
    for (int i = 0; i < t.size; ++i) {
        if (nelems[i] > (size_t)-1 / sizeof(T)) return ISHMEM_ERR_ARG;
        bytes[i] = nelems[i] * sizeof(T);
    }
    return ishmem_collectmem(team, dest, src, bytes);
}
#define ISHMEMI_DEF_COLL(NAME, T)                                                                                   \
    extern "C" int ishmem_##NAME##_broadcast(ishmem_team_t team, T *dest, const T *src, size_t nelems, int root)     \
    {                                                                                                                \
        if (((uintptr_t)dest | (uintptr_t)src) % sizeof(T)) return ISHMEM_ERR_ALIGN;                                 \
        if (nelems > (size_t)-1 / sizeof(T)) return ISHMEM_ERR_ARG;                                                  \
        return ishmem_broadcastmem(team, dest, src, nelems * sizeof(T), root);                                       \
    }                                                                                                                \
    extern "C" int ishmem_##NAME##_fcollect(ishmem_team_t team, T *dest, const T *src, size_t nelems)                \
    {                                                                                                                \
        if (((uintptr_t)dest | (uintptr_t)src) % sizeof(T)) return ISHMEM_ERR_ALIGN;                                 \
        if (nelems > (size_t)-1 / sizeof(T)) return ISHMEM_ERR_ARG;                                                  \
        return ishmem_fcollectmem(team, dest, src, nelems * sizeof(T));                                              \
    }                                                                                                                \
    extern "C" int ishmem_##NAME##_collect(ishmem_team_t team, T *dest, const T *src, const size_t *nelems)          \
    {                                                                                                                \
        return typed_collect<T>(team, dest, src, nelems);                                                            \
    }                                                                                                                \
    extern "C" int ishmem_##NAME##_alltoall(ishmem_team_t team, T *dest, const T *src, size_t nelems)                \
    {                                                                                                                \
        if (((uintptr_t)dest | (uintptr_t)src) % sizeof(T)) return ISHMEM_ERR_ALIGN;                                 \
        if (nelems > (size_t)-1 / sizeof(T)) return ISHMEM_ERR_ARG;                                                  \
        return ishmem_alltoallmem(team, dest, src, nelems * sizeof(T));                                              \
    }
ISHMEMI_DEF_COLL(float, float)
ISHMEMI_DEF_COLL(double, double)
ISHMEMI_DEF_COLL(int, int)
ISHMEMI_DEF_COLL(long, long)
ISHMEMI_DEF_COLL(int32, int32_t)
ISHMEMI_DEF_COLL(int64, int64_t)
ISHMEMI_DEF_COLL(uint8, uint8_t)
ISHMEMI_DEF_COLL(uint32, uint32_t)
ISHMEMI_DEF_COLL(uint64, uint64_t)

extern "C" int ishmemx_reduce(ishmem_team_t team, void *dest, const void *src, size_t nreduce, int op, int dtype,
                              int algorithm)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    ishmemi_team t;
    int rc = team_of(team, &t);
    if (rc) return rc;
    const size_t es = dtype_size(dtype);
    reduce_kernel_t k = pick_reduce(op, dtype);
    if (!es || !k) return ISHMEM_ERR_ARG;
    if (algorithm < ISHMEMX_REDUCE_AUTO || algorithm > ISHMEMX_REDUCE_SPLIT) return ISHMEM_ERR_ARG;
    if (((uintptr_t)dest | (uintptr_t)src) % es) return ISHMEM_ERR_ALIGN;
    if (nreduce > (size_t)-1 / es) return ISHMEM_ERR_ARG;
    const size_t bytes = nreduce * es;
    if ((rc = check_sym2(dest, bytes, src, bytes))) return rc;
    const char *d = (const char *)dest, *sp = (const char *)src;
    const bool overlap = d < sp + bytes && sp < d + bytes;
    if (algorithm == ISHMEMX_REDUCE_AUTO) algorithm = ISHMEMX_REDUCE_SPLIT;
    /* in place is fine when each element is read from all sources and written to all dests by
     * one thread (split); any other overlap would mix old and new values */
    if (overlap && !(d == sp && algorithm == ISHMEMX_REDUCE_SPLIT)) return ISHMEM_ERR_ARG;
    cudaStream_t s;
    if ((rc = ishmemi_team_stream_begin(team, &s))) return rc;
    if (nreduce) {
        coll_args a = {};
        a.team = team;
        a.dest = (char *)dest;
        a.src = sp;
        a.n = nreduce;
        a.duplicated = (algorithm == ISHMEMX_REDUCE_DUPLICATED);
        const size_t per_member = a.duplicated ? bytes : bytes / t.size + 1;
        /* loads/stores, one tile of threads x tile_vpt vectors per block (blocks start in index
         * order, so the running blocks sweep one contiguous window of every source and
         * destination).  Small inputs take one vector per thread, so that a few hundred KiB
         * already occupy every SM; large ones two. */
        int threads = g.coll_threads > 512 ? 512 : g.coll_threads;
        a.tile_vpt = 2;
        const size_t nvec = (bytes + 15) / 16;
        if (g.coll_groups > 0) {
            a.groups = g.coll_groups;
        } else {
            threads = threads > 128 ? 128 : threads;
            if (nvec <= (size_t)g.sm_count * 4 * 128 * (a.duplicated ? t.size : 1)) a.tile_vpt = 1;
            size_t blocks = (nvec + (size_t)threads * a.tile_vpt - 1) / ((size_t)threads * a.tile_vpt);
            /* the grid is groups x members blocks (in the duplicated form each member's `groups`
             * blocks sweep all tiles, so the tiles per block come out the same) */
            blocks = (blocks + t.size - 1) / t.size;
            const size_t most = (size_t)0x7fffffff / (size_t)t.size;
            a.groups = (int)(blocks < 1 ? 1 : (blocks < most ? blocks : most));
        }
        /* ISHMEMX_OPT_REDUCE_BULK selects the TMA fold ring instead (one resident block per SM, three
         * stages of P tiles in shared memory): 6.2 TB/s at 12 PEs x 256 MiB where the tiles above
         * reach 6.5. */
        const bool use_bulk = g.opt[ISHMEMX_OPT_REDUCE_BULK] != 0 && !a.duplicated;
        if (use_bulk && g.coll_groups == 0 && per_member >= (1u << 20) && t.size <= 48) {
            unsigned want = 192 * 1024 + 128;
            if (want > g.max_dyn_smem) want = (unsigned)g.max_dyn_smem;
            if (cudaFuncSetAttribute((const void *)k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)want) ==
                cudaSuccess) {
                a.staging_bytes = want;
                size_t cap = (size_t)g.sm_count / t.size, need = (per_member + (256u << 10) - 1) / (256u << 10);
                if (cap < 1) cap = 1;
                a.groups = (int)(need < cap ? need : cap);
                threads = 512;
            }
        }
        k<<<a.groups * t.size, threads, a.staging_bytes, s>>>(g.d_ctx, a);
        ishmemi_count_launch();
        rc = ishmemi_check_launch("k_reduce");
    }
    ishmemi_team_stream_end();
    return rc;
}

#define ISHMEMI_DEF_REDUCE(NAME, T, OPNAME, OP, DT)                                                          \
    extern "C" int ishmem_##NAME##_##OPNAME##_reduce(ishmem_team_t team, T *dest, const T *src, size_t nreduce) \
    {                                                                                                        \
        return ishmemx_reduce(team, dest, src, nreduce, OP, DT, ISHMEMX_REDUCE_AUTO);                        \
    }
#define ISHMEMI_DEF_REDUCE_ARITH(NAME, T, DT)                                                 \
    ISHMEMI_DEF_REDUCE(NAME, T, sum, ISHMEM_OP_SUM, DT) ISHMEMI_DEF_REDUCE(NAME, T, max, ISHMEM_OP_MAX, DT) \
    ISHMEMI_DEF_REDUCE(NAME, T, min, ISHMEM_OP_MIN, DT) ISHMEMI_DEF_REDUCE(NAME, T, prod, ISHMEM_OP_PROD, DT)
#define ISHMEMI_DEF_REDUCE_BITS(NAME, T, DT)                                                  \
    ISHMEMI_DEF_REDUCE(NAME, T, and, ISHMEM_OP_AND, DT) ISHMEMI_DEF_REDUCE(NAME, T, or, ISHMEM_OP_OR, DT) \
    ISHMEMI_DEF_REDUCE(NAME, T, xor, ISHMEM_OP_XOR, DT)
ISHMEMI_DEF_REDUCE_ARITH(int32, int32_t, ISHMEM_T_INT32)
ISHMEMI_DEF_REDUCE_ARITH(int64, int64_t, ISHMEM_T_INT64)
ISHMEMI_DEF_REDUCE_ARITH(uint32, uint32_t, ISHMEM_T_UINT32)
ISHMEMI_DEF_REDUCE_ARITH(uint64, uint64_t, ISHMEM_T_UINT64)
ISHMEMI_DEF_REDUCE_ARITH(float, float, ISHMEM_T_FLOAT)
ISHMEMI_DEF_REDUCE_ARITH(double, double, ISHMEM_T_DOUBLE)
ISHMEMI_DEF_REDUCE_BITS(int32, int32_t, ISHMEM_T_INT32)
ISHMEMI_DEF_REDUCE_BITS(int64, int64_t, ISHMEM_T_INT64)
ISHMEMI_DEF_REDUCE_BITS(uint32, uint32_t, ISHMEM_T_UINT32)
ISHMEMI_DEF_REDUCE_BITS(uint64, uint64_t, ISHMEM_T_UINT64)
ISHMEMI_DEF_REDUCE_ARITH(int8, int8_t, ISHMEM_T_INT8)
ISHMEMI_DEF_REDUCE_ARITH(uint8, uint8_t, ISHMEM_T_UINT8)
ISHMEMI_DEF_REDUCE_ARITH(int16, int16_t, ISHMEM_T_INT16)
ISHMEMI_DEF_REDUCE_ARITH(uint16, uint16_t, ISHMEM_T_UINT16)
ISHMEMI_DEF_REDUCE_BITS(int8, int8_t, ISHMEM_T_INT8)
ISHMEMI_DEF_REDUCE_BITS(uint8, uint8_t, ISHMEM_T_UINT8)
ISHMEMI_DEF_REDUCE_BITS(int16, int16_t, ISHMEM_T_INT16)
ISHMEMI_DEF_REDUCE_BITS(uint16, uint16_t, ISHMEM_T_UINT16)

extern "C" int ishmemx_collective_on_device(int which, ishmem_team_t team, void *dest, const void *src, size_t n,
                                            int root, int op, int dtype, int threads, int repeat)
{
    auto &g = g_ishmem;
    ISHMEMI_REQUIRE_INIT();
    ishmemi_team t;
    int rc = team_of(team, &t);
    if (rc) return rc;
    if (which < 0 || which > 5 || threads < 32 || threads > 1024 || repeat < 1) return ISHMEM_ERR_ARG;
    if (which != 3) {
        size_t es = 1;
        if (which == 2) {
            es = dtype_size(dtype);
            if (!es || !pick_reduce(op, dtype)) return ISHMEM_ERR_ARG;
            if (((uintptr_t)dest | (uintptr_t)src) % es) return ISHMEM_ERR_ALIGN;
        }
        if (which == 0 && (root < 0 || root >= t.size)) return ISHMEM_ERR_INVALID_PE;
        if (n > (size_t)-1 / (es * t.size)) return ISHMEM_ERR_ARG;
        size_t sbytes = (which == 4 ? n * t.size : n * es), dbytes = (which == 1 || which == 4 || which == 5) ? n * es * t.size : sbytes;
        if ((rc = check_sym2(dest, dbytes, src, sbytes))) return rc;
        const char *d = (const char *)dest, *sp = (const char *)src;
        if (d < sp + sbytes && sp < d + dbytes) return ISHMEM_ERR_ARG;
    }
    cudaStream_t s;
    if ((rc = ishmemi_team_stream_begin(team, &s))) return rc;
    coll_args a = {};
    a.team = team;
    a.dest = (char *)dest;
    a.src = (const char *)src;
    a.n = n;
    a.root = root;
    a.repeat = repeat;
    const ishmem_ctx_t *ctxs = g.d_ctx;
    void *params[] = {(void *)&ctxs, (void *)&a};
    rc = ishmemi_cuda(cudaLaunchCooperativeKernel((void *)pick_dev(which, op, dtype), dim3(t.size), dim3(threads),
                                                  params, 0, s),
                      "cudaLaunchCooperativeKernel(collective)");
    ishmemi_count_launch();
    ishmemi_team_stream_end();
    return rc;
}
