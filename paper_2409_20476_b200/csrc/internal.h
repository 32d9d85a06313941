/* Host-side state of libishmem.so, shared by its translation units.  Not part of the ABI. */
#ifndef ISHMEMI_INTERNAL_H
#define ISHMEMI_INTERNAL_H

#include <cuda_runtime.h>

#include <map>
#include <mutex>
#include <string>

#include "ishmem.h"
#include "ishmem_device.cuh"

#define ISHMEMI_ALIGN 256u

struct ishmemi_state {
    bool initialised = false;
    int device = 0;
    int npes = 0;
    size_t heap_bytes = 0;
    char *base = nullptr;       /* npes consecutive slices */
    bool owns_heap = false;
    ishmem_ctx_t *d_ctx = nullptr; /* device array of npes contexts */
    ishmem_ctx_t h_ctx[ISHMEM_MAX_PES];
    char *d_internal = nullptr; /* npes * ISHMEMI_INTERNAL_BYTES, then the status word */
    int *d_status = nullptr;
    void *h_pinned = nullptr;   /* small pinned scratch for values returned to the host */

    /* streams: one per PE, one for team-wide launches, one copy-engine side stream per PE */
    cudaStream_t pe_stream[ISHMEM_MAX_PES] = {};
    bool owns_pe_stream[ISHMEM_MAX_PES] = {};
    cudaStream_t engine_stream[ISHMEM_MAX_PES] = {};
    cudaStream_t team_stream = nullptr;
    bool owns_team_stream = false;
    cudaEvent_t ev_pe[ISHMEM_MAX_PES] = {};     /* last recorded point of each PE stream */
    cudaEvent_t ev_engine[ISHMEM_MAX_PES] = {};
    cudaEvent_t ev_team = nullptr;
    /* lazy cross-stream ordering: a PE stream is "dirty" when it has work the team stream
     * has not waited for; team_seq counts team launches, pe_seen_team[p] the last one PE
     * p's stream has waited for */
    bool pe_dirty[ISHMEM_MAX_PES] = {};
    bool nbi_pending[ISHMEM_MAX_PES] = {};
    unsigned long long team_seq = 0;
    unsigned long long team_event_seq = 0; /* team_seq value ev_team was last recorded for */
    unsigned long long pe_seen_team[ISHMEM_MAX_PES] = {};

    /* symmetric allocator: offset -> size of free and of used blocks */
    std::map<size_t, size_t> free_blocks, used_blocks;

    ishmemi_team teams[ISHMEM_MAX_TEAMS] = {};
    size_t cutover[3] = {0, 0, 0};
    size_t cutover_put_upto = (size_t)-1; /* host-initiated put/get use the engine for cutover[0] <= n < this */
    size_t wg_cutover = (size_t)-1; /* device-initiated work-group put/get: bytes from which the engine is used */
    size_t hybrid_head = 0;         /* ... and bytes of the head the group copies itself meanwhile */
    long long opt[ISHMEMX_OPT_COUNT] = {}; /* ishmemx_set_option: launch-shape switches */
    int coll_groups = 0, coll_threads = 512;
    int bcast_root_dest = 1;
    unsigned long long wait_limit_ns = 2000000000ull;
    int sm_count = 148;
    size_t max_dyn_smem = 0;
    unsigned long long launches = 0; /* kernels launched by the library */
    std::string last_cuda_error;
    std::mutex mu;
};

extern ishmemi_state g_ishmem;

/* status of a CUDA call; records the message on failure */
int ishmemi_cuda(cudaError_t e, const char *what);
#define ISHMEMI_CUDA(call)                                   \
    do {                                                     \
        int rc__ = ishmemi_cuda((call), #call);              \
        if (rc__) return rc__;                               \
    } while (0)
#define ISHMEMI_REQUIRE_INIT()                                        \
    do {                                                              \
        if (!g_ishmem.initialised) return ISHMEM_ERR_NOT_INITIALIZED; \
    } while (0)

/* Offset of a symmetric address (PE 0's copy) or -1 if [p, p+n) is not inside PE 0's slice. */
long long ishmemi_sym_offset(const void *p, size_t n);
/* my_pe's local address of `p` if p is symmetric, else p itself (a private device pointer) */
char *ishmemi_localise(const void *p, size_t n, int my_pe);
int ishmemi_check_pe(int pe);
/* stream ordering helpers */
cudaStream_t ishmemi_pe_stream_for_op(int pe);   /* joins the team stream first if needed */
int ishmemi_team_stream_begin(ishmem_team_t team, cudaStream_t *out); /* waits for dirty members */
void ishmemi_team_stream_end();
void ishmemi_push_ctx();                         /* re-upload host contexts to the device */
void ishmemi_count_launch(unsigned n = 1);
int ishmemi_check_launch(const char *what);      /* cudaGetLastError -> status */
int ishmemi_engine_copy(int my_pe, void *dst, const void *src, size_t n, bool blocking);
/* reverse-offload proxy (proxy.cu) */
void ishmemi_proxy_finalize();
void ishmemi_proxy_set_cutover(size_t nbytes, size_t hybrid_head);

#endif
