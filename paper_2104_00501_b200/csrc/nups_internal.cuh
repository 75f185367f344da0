// Internal declarations shared by the translation units of libnups.so.
// Device helpers are inline; nothing here is exported.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/nups.h"

#define NUPS_MAX_DISTS 64
#define NUPS_MAX_HANDLES 256
#define NUPS_LOCAL_PROBES 64
#define NUPS_OWNER_DEFAULT 255
#define NUPS_INVALID_KEY 0xFFFFFFFFu
#define NUPS_MAX_POOL 1024
#define NUPS_MAX_TIMED 65536
#define NUPS_TIMED_KINDS 8
#define NUPS_MAX_STEP_BLOCKS 8192
#define NUPS_SAMPLE_AHEAD 16

// ---------------------------------------------------------------------------------------------
// Device-resident status and statistics
// ---------------------------------------------------------------------------------------------
struct DevStat {
    int status;                        // first device-detected error, 0 = none
    int pad;
    unsigned long long hot_hits;       // accesses served by a replica
    unsigned long long cold_hits;      // accesses served in place
    unsigned long long unused0;
    unsigned long long tmp[4];
    // gradient-norm clipping of replicated-key updates: norms applied by finished steps, and by the running one
    double clip_sum;
    unsigned long long clip_cnt;
    double clip_step_sum;
    unsigned long long clip_step_cnt;
};

// What kernels need to know about a store; passed by value.
struct View {
    float* val;
    float* acc;
    float* dval;               // [R][Hcap][L] pending replica updates of the value table
    float* dacc;               // same for the accumulator table
    const uint32_t* hot_bits;  // one bit per key: replicated?
    const int32_t* slot_of;    // key -> hot slot (>= 0) or negative
    uint32_t* dirty;           // [R][Hcap] worker's replica of the slot touched since last sync
    unsigned long long* cnt;   // [num_keys] access counts
    uint32_t* own;             // [num_keys] ownership words (see mark_localize); NULL = not tracked
    DevStat* st;
    double* loss_partial;      // [4 * NUPS_MAX_STEP_BLOCKS] per-warp loss sums of the running step kernel
    uint64_t num_keys;
    uint64_t Hcap;
    uint32_t H;
    uint32_t L4;               // floats per row / 4
    uint32_t R;
    uint32_t count;            // count accesses?
    uint32_t merge_mean;       // merges add the mean over the workers that touched a slot, not the sum
    uint32_t f64;              // values are doubles (rows are still counted in 16-byte chunks, L4)
    uint32_t epoch_tag;        // number of the running call, shifted into the upper 24 bits of an ownership word
    float clip_factor;         // > 0: updates to replicated keys are clipped at this multiple of their mean norm
};

struct Dist {
    int used, uniform, level;
    uint32_t key_base, U, G;
    uint64_t n, W, seed;
    void* table;               // AliasEntry[n]
    unsigned long long* off;   // device [2][R]: next unused position of each worker's stream; a call reads
                               // half `cur` and writes the other half, then the host flips `cur`
    int cur;
};

struct AliasEntry {
    unsigned long long thr;
    uint32_t alias;
    uint32_t pad;
};

struct Handle {
    int used, dist;
    uint64_t N, cursor;
    char* buf;                 // device buffer, kept for reuse after release
    size_t cap;
};

struct nups_store {
    uint64_t num_keys;
    uint32_t L, R;             // L = row length in 4-byte units (value_len for fp32 values, 2 * value_len for fp64 values)
    uint32_t value_len, vb;    // values per row; bytes per value (4 or 8)
    nups_config cfg;
    float *val, *acc;
    uint32_t* hot_bits;
    int32_t* slot_of;
    uint32_t* hot_keys;
    uint64_t H, Hcap;
    float *dval, *dacc;
    uint32_t* dirty;
    unsigned long long* cnt;
    uint32_t* own;
    uint32_t epoch;            // calls that moved keys so far (24 bits, see nups_new_epoch)
    DevStat* st;
    double* loss_partial;
    char* scratch;
    size_t scratch_bytes;
    size_t dev_bytes, dev_cap; // device memory held by the store, and its limit (0 = none)
    uint32_t* negs_buf;        // negatives drawn for the workload steps, possibly several batches ahead
    uint64_t negs_cap;
    uint32_t* last_negs;       // the slice of negs_buf that the most recent step used
    uint64_t last_negs_n;
    int ahead_dist;            // sample-ahead state: batches [ahead_next, ahead_total) of ahead_N samples
    uint64_t ahead_N;          // from ahead_dist are drawn but not handed out yet (-1 = none)
    uint32_t ahead_total, ahead_next;
    uint64_t steps, syncs, launches;
    int device, sm_count, max_smem;
    int timing;                // record events around the main kernels?
    cudaEvent_t* ev;           // [2 * NUPS_MAX_TIMED] begin/end pairs
    unsigned char* ev_kind;    // [NUPS_MAX_TIMED] which kernel the pair brackets (NUPS_TIMED_*)
    uint32_t ev_n;             // pairs recorded since the last query
    double ev_ms[NUPS_TIMED_KINDS];          // time of the pairs folded in so far, by kind
    uint64_t ev_launches[NUPS_TIMED_KINDS];
    struct nups_background* bg; // time-based replica synchronisation (background.cu); NULL = never started
    cudaStream_t side;          // nups_run_sgns: a due replica merge runs here, beside the next steps' sample draw
    cudaEvent_t side_fork, side_join;
    bool push_smem_opted, complex_smem_opted[2][2][2][2];   // large dynamic shared memory asked for on this store's device
    float* merge_snap[2];       // merging across GPUs (shard.cu): each table as all GPUs last agreed on it; NULL = never marked
    Dist dist[NUPS_MAX_DISTS];
    Handle handle[NUPS_MAX_HANDLES];
};

// ---------------------------------------------------------------------------------------------
// Host helpers
// ---------------------------------------------------------------------------------------------
extern thread_local char g_nups_cuda_err[256];
nups_status nups_cuda_fail(cudaError_t e, const char* what);

#define CK(call)                                                   \
    do {                                                           \
        cudaError_t e__ = (call);                                  \
        if (e__ != cudaSuccess) return nups_cuda_fail(e__, #call); \
    } while (0)

#define LAUNCH_CHECK(store)                                         \
    do {                                                            \
        (store)->launches++;                                        \
        cudaError_t e__ = cudaGetLastError();                       \
        if (e__ != cudaSuccess) return nups_cuda_fail(e__, "kernel launch"); \
    } while (0)

static inline unsigned grid_for(uint64_t work, unsigned per_block, unsigned cap = 0x7FFFFFFFu)
{
    uint64_t g = (work + per_block - 1) / per_block;
    if (g < 1) g = 1;
    if (g > cap) g = cap;
    return (unsigned)g;
}

View nups_view(const nups_store* s);
// kinds of kernels that nups_kernel_timing brackets (index into the arrays nups_kernel_times returns)
enum { NUPS_TIMED_PULL = 0, NUPS_TIMED_PUSH = 1, NUPS_TIMED_STEP = 2, NUPS_TIMED_SAMPLE_ROWS = 3, NUPS_TIMED_DRAW = 4 };
void nups_time_begin(nups_store* s, cudaStream_t st, int kind);
void nups_time_end(nups_store* s, cudaStream_t st);
nups_status nups_scratch(nups_store* s, size_t bytes, char** out);     // grow-only scratch, 256-byte aligned
// Device memory of a store goes through these two so that the store's own limit can refuse a request before the
// allocator is asked.  nups_dev_alloc leaves *p null on failure.
nups_status nups_dev_alloc(nups_store* s, void** p, size_t bytes);
void nups_dev_free(nups_store* s, void* p, size_t bytes);
nups_status nups_new_epoch(nups_store* s, cudaStream_t st);          // call before taking the view of a call that moves keys

// Programmatic dependent launch.  A kernel started through nups_launch_dependent may become resident while the kernel
// before it on the stream is still draining its last blocks, which hides the launch latency between the back-to-back
// kernels of a training loop.  Such a kernel calls grid_dependency_wait() before its first access to global memory: the
// wait returns once every earlier kernel of the stream has finished and its writes are visible, so the order of the
// stream's work is what it is with a plain launch.  The call is a no-op in a kernel that was launched the plain way.
// It also lets the NEXT kernel of the stream become resident early; that one can only start once every block of this
// kernel has been scheduled, so the blocks waiting there never take a place that this kernel still needs.
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");
}

template <class... KArgs, class... Args>
static inline cudaError_t nups_launch_dependent(void (*kernel)(KArgs...), dim3 grid, unsigned block, size_t smem,
                                                cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

// background.cu
nups_status nups_background_start(nups_store* s, uint32_t period_us);
void nups_background_stop(nups_store* s);
void nups_background_begin(nups_store* s, cudaStream_t st);
void nups_background_end(nups_store* s, cudaStream_t st);
uint64_t nups_background_merges(nups_store* s);

// primitives.cu
size_t nups_scan_scratch_bytes(uint64_t n);
size_t nups_sort_scratch_bytes(uint64_t n);
// Exclusive prefix sum of n uint64 values (in place allowed); *d_total (device, nullable) receives the sum.
nups_status nups_scan_u64(nups_store* s, const unsigned long long* d_in, unsigned long long* d_out, uint64_t n,
                          unsigned long long* d_total, char* scratch, cudaStream_t st);
// Stable LSD radix sort of (key, value) pairs on the low `bits` bits; result ends up in (k_out, v_out).
nups_status nups_sort_pairs(nups_store* s, unsigned long long* k_in, uint32_t* v_in, unsigned long long* k_out,
                            uint32_t* v_out, uint64_t n, int bits, char* scratch, cudaStream_t st);

// store.cu internals used by steps.cu / sampling.cu
// (value buffers are passed as float* whatever the value type: storage, counted in 4-byte units)
nups_status nups_push_internal(nups_store* s, const uint32_t* d_keys, uint64_t n_rows, uint32_t rows_per_item,
                               const float* d_dval, const float* d_dacc, cudaStream_t st);
size_t nups_push_scratch_bytes(const nups_store* s, uint64_t n_rows);
nups_status nups_push_with_scratch(nups_store* s, const uint32_t* d_keys, uint64_t n_rows, uint32_t rows_per_item,
                                   const float* d_dval, const float* d_dacc, char* scratch, cudaStream_t st);
nups_status nups_gather_internal(nups_store* s, const uint32_t* d_keys, uint64_t n, float* d_out_val,
                                 float* d_out_acc, int worker_map, uint64_t map_base, uint64_t map_total,
                                 int do_count, cudaStream_t st,
                                 uint32_t* d_keys_copy /* nullable: also write the keys here */);
nups_status nups_sync_internal(nups_store* s, cudaStream_t st);
// sampling.cu internals used by steps.cu
nups_status nups_draw_negatives(nups_store* s, int32_t dist, uint64_t N, cudaStream_t st);
nups_status nups_sample_ahead_rewind(nups_store* s, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// Device helpers
// ---------------------------------------------------------------------------------------------
#ifdef __CUDACC__

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                              uint32_t k1, uint32_t out[4])
{
    // Philox4x32-10 (Salmon et al., SC'11): ten rounds, each two 32x32->64 multiplies with the
    // halves crossed and xor-ed with the round key; the key advances by the Weyl constants.
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Counter layout of every draw: (index lo, index hi, stream, purpose + 256 * block).
__device__ __forceinline__ void philox_at(uint64_t seed, uint64_t index, uint32_t stream, uint32_t purpose,
                                          uint32_t block, uint32_t out[4])
{
    philox4x32_10((uint32_t)index, (uint32_t)(index >> 32), stream, purpose + 256u * block, (uint32_t)seed,
                  (uint32_t)(seed >> 32), out);
}

// Worker of item i of n: contiguous chunks, floor(i * R / n).
__device__ __forceinline__ uint32_t worker_of_item(uint64_t i, uint64_t n, uint32_t R)
{
    if (R == 1) return 0;
    if (((n * R) >> 32) == 0) return ((uint32_t)i * R) / (uint32_t)n;   // the usual case: a 32-bit division
    return (uint32_t)((i * R) / n);          // calls take fewer than 2^32 items: i * R < 2^40
}

// First item of worker q's chunk: the smallest i with floor(i * R / n) >= q, i.e. ceil(q * n / R).  A loop whose
// item index only grows keeps its worker and the next chunk's first item instead of dividing for every item.
__device__ __forceinline__ uint64_t worker_first_item(uint32_t q, uint64_t n, uint32_t R)
{
    return ((uint64_t)q * n + R - 1) / R;
}

// Sub-handle boundaries of a handle of N samples: b_q = floor(q * N / R).
__device__ __forceinline__ uint64_t chunk_begin(uint32_t q, uint64_t N, uint32_t R) { return ((uint64_t)q * N) / R; }
__device__ __forceinline__ uint32_t chunk_of_pos(uint64_t pos, uint64_t N, uint32_t R)
{
    if (R == 1) return 0;
    uint32_t q = (uint32_t)((pos * R) / N);
    if (q >= R) q = R - 1;
    while (q + 1 < R && chunk_begin(q + 1, N, R) <= pos) ++q;
    while (q > 0 && chunk_begin(q, N, R) > pos) --q;
    return q;
}

// worker_map: 0 = items of a call (floor(i*R/n), i = (base + idx) / rows_per_item handled by caller),
//             1 = positions of a sample handle (sub-handle chunks)
__device__ __forceinline__ uint32_t worker_by_map(int map, uint64_t idx, uint64_t total, uint32_t R)
{
    return map == 0 ? worker_of_item(idx, total, R) : chunk_of_pos(idx, total, R);
}

__device__ __forceinline__ bool key_is_hot(const View& v, uint32_t k)
{
    return v.H != 0 && ((__ldg(v.hot_bits + (k >> 5)) >> (k & 31)) & 1u);
}

// Ownership word of a key: low byte = owning worker (NUPS_OWNER_DEFAULT = never moved: key mod R),
// upper 24 bits = number of the call that wrote it.
__device__ __forceinline__ bool word_is_local(uint32_t word, uint32_t q, uint32_t k, uint32_t R)
{
    const uint32_t o = word & 0xFFu;
    return (o == NUPS_OWNER_DEFAULT ? k % R : o) == q;
}

__device__ __forceinline__ bool key_is_local(const View& v, uint32_t q, uint32_t k)
{
    if (key_is_hot(v, k)) return true;
    if (!v.own) return true;
    return word_is_local(v.own[k], q, k, v.R);
}

// mark a replica slot as touched without waiting for anything to come back
__device__ __forceinline__ void mark_dirty(const View& v, uint32_t q, int slot)
{
    asm volatile("red.global.or.b32 [%0], 1;" ::"l"(v.dirty + (size_t)q * v.Hcap + slot) : "memory");
}
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// Move key -> worker q (the paper's localize).  Requests of one call take effect when the call ends
// and the last one wins; callers visit workers in ascending order, so the largest requesting worker
// gets the key.  Nothing reads ownership while a call that moves keys runs, so the word can be
// written at once: the call's number sits above the worker, hence one atomic maximum both replaces
// whatever an earlier call left and keeps the largest worker of this call.  Replicated keys are
// local to every worker and never move, which also keeps the hottest keys from queueing at one
// address; a word that already shows this call and a worker >= q needs no atomic.
__device__ __forceinline__ void mark_localize(const View& v, uint32_t key, uint32_t q)
{
    if (key_is_hot(v, key)) return;
    const uint32_t want = v.epoch_tag | q;
    if (__ldcg(v.own + key) >= want) return;
    atomicMax(v.own + key, want);
}

// The same for the keys of independent draws, which rarely repeat: reading the word first would add one more
// scattered memory access per sample (these kernels are bound by the rate of such accesses).  `repeats` = the key
// shows up more than once among the warp's samples, the sign of a very frequent key: those still look first, so that
// a frequent key that is not replicated does not queue thousands of atomics at one address.
__device__ __forceinline__ void mark_localize_rare(const View& v, uint32_t key, uint32_t q, bool repeats)
{
    if (key_is_hot(v, key)) return;
    const uint32_t want = v.epoch_tag | q;
    if (repeats && __ldcg(v.own + key) >= want) return;
    atomicMax(v.own + key, want);
}

__device__ __forceinline__ void flag_bad_key(const View& v) { atomicCAS(&v.st->status, 0, NUPS_EKEY); }

__device__ __forceinline__ void red_add_v4(float* addr, float4 x)
{
    // one 128-bit reduction to global memory, no return value
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(x.x), "f"(x.y), "f"(x.z), "f"(x.w)
                 : "memory");
}

__device__ __forceinline__ float4 ld_stream_v4(const float4* p)
{
    float4 r;
    asm volatile("ld.global.cs.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ void st_stream_v4(float4* p, float4 x)
{
    asm volatile("st.global.cs.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(x.x), "f"(x.y), "f"(x.z), "f"(x.w)
                 : "memory");
}

// 256-bit global loads and stores (sm_100): 32-byte aligned addresses
struct F8 { float4 a, b; };
__device__ __forceinline__ F8 ld8_cached(const float* p)
{
    F8 r;
    asm volatile("ld.global.nc.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r.a.x), "=f"(r.a.y), "=f"(r.a.z), "=f"(r.a.w), "=f"(r.b.x), "=f"(r.b.y), "=f"(r.b.z), "=f"(r.b.w) : "l"(p));
    return r;
}
__device__ __forceinline__ F8 ld8_stream(const float* p)
{
    F8 r;
    asm volatile("ld.global.cs.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r.a.x), "=f"(r.a.y), "=f"(r.a.z), "=f"(r.a.w), "=f"(r.b.x), "=f"(r.b.y), "=f"(r.b.z), "=f"(r.b.w) : "l"(p));
    return r;
}
__device__ __forceinline__ F8 ld8_plain(const float* p)
{
    F8 r;
    asm volatile("ld.global.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r.a.x), "=f"(r.a.y), "=f"(r.a.z), "=f"(r.a.w), "=f"(r.b.x), "=f"(r.b.y), "=f"(r.b.z), "=f"(r.b.w) : "l"(p));
    return r;
}
__device__ __forceinline__ void st8_stream(float* p, const F8& r)
{
    asm volatile("st.global.cs.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(r.a.x), "f"(r.a.y), "f"(r.a.z),
                 "f"(r.a.w), "f"(r.b.x), "f"(r.b.y), "f"(r.b.z), "f"(r.b.w) : "memory");
}

__device__ __forceinline__ float4 add4(float4 a, float4 b) { return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w); }

// A 16-byte chunk of a row holds four floats or two doubles; kernels that only move rows do not care, kernels that add
// (replica reads, pushes, merges) take the value type as a template argument.
__device__ __forceinline__ double2 as_d2(float4 a)
{
    return make_double2(__hiloint2double(__float_as_int(a.y), __float_as_int(a.x)),
                        __hiloint2double(__float_as_int(a.w), __float_as_int(a.z)));
}
__device__ __forceinline__ float4 as_f4(double2 d)
{
    return make_float4(__int_as_float(__double2loint(d.x)), __int_as_float(__double2hiint(d.x)),
                       __int_as_float(__double2loint(d.y)), __int_as_float(__double2hiint(d.y)));
}
template <bool F64>
__device__ __forceinline__ float4 add_chunk(float4 a, float4 b)
{
    if (F64) {
        const double2 x = as_d2(a), y = as_d2(b);
        return as_f4(make_double2(x.x + y.x, x.y + y.y));
    }
    return add4(a, b);
}
template <bool F64>
__device__ __forceinline__ void red_add_chunk(float* addr, float4 x)
{
    if (F64) {
        const double2 d = as_d2(x);
        asm volatile("red.global.add.f64 [%0], %1;" ::"l"(addr), "d"(d.x) : "memory");
        asm volatile("red.global.add.f64 [%0], %1;" ::"l"(addr + 2), "d"(d.y) : "memory");
    } else {
        red_add_v4(addr, x);
    }
}

__device__ __forceinline__ float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
    return x;
}

#endif  // __CUDACC__
