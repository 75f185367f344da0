// shard.cu - a value table partitioned over several GPUs by key range and accessed through peer memory.
//
// Section 3.1 of the paper: a parameter server partitions the parameters over its servers (the classic scheme: by key
// range) and a worker reaches a parameter that another node holds by sending that node a message.  Between GPUs of one
// NVLink / NVSwitch domain there is nothing to send: a peer's HBM is addressable, so "remote access" is a load from, or
// a floating-point reduction into, the owner's memory, issued by the very kernel that moves the caller's rows.  Shard j
// holds the rows of keys [j * keys_per_shard, (j + 1) * keys_per_shard); every process keeps its own shard and the base
// addresses of the others' (same-process pointers, or CUDA IPC mappings of another process's allocation).  pull gathers
// rows from wherever they live, push adds to them there; the owner takes no part, and there is no exchange of keys
// first.  Replication of hot keys is a matter of the single-GPU store (store.cu); this file is the partitioned,
// non-replicated part.
#include "nups_internal.cuh"

#include <cstdio>
#include <cstdlib>
#include <cstring>

struct nups_shard_table {
    uint64_t num_keys, keys_per_shard;
    uint32_t value_len, n_shards, my_shard;
    int device;
    float* local;                               // this process's shard [keys_per_shard][value_len], owned
    float* base_h[NUPS_MAX_SHARDS];             // every shard's first row as this process addresses it (null = not attached)
    void* ipc_opened[NUPS_MAX_SHARDS];          // mappings opened here, closed on destroy
    float** base_d;                             // the same addresses on the device
    int* status_d;                              // device status word: 0 or NUPS_EKEY
    bool bases_changed;
    char err[160];
};

static nups_status shard_fail(nups_shard_table* t, cudaError_t e, const char* what)
{
    if (t) snprintf(t->err, sizeof(t->err), "%s: %s", what, cudaGetErrorString(e));
    cudaGetLastError();
    return NUPS_ECUDA;
}
#define SCK(t, call)                                                     \
    do {                                                                 \
        cudaError_t e__ = (call);                                        \
        if (e__ != cudaSuccess) return shard_fail((t), e__, #call);      \
    } while (0)

extern "C" nups_status nups_shard_table_create(uint64_t num_keys, uint32_t value_len, uint32_t n_shards, uint32_t my_shard,
                                               nups_shard_table** out)
{
    if (!out) return NUPS_EINVAL;
    *out = nullptr;
    if (num_keys == 0 || num_keys > 0xFFFFFFFFull || value_len == 0 || (value_len & 3) || n_shards == 0 ||
        n_shards > NUPS_MAX_SHARDS || my_shard >= n_shards)
        return NUPS_EINVAL;
    nups_shard_table* t = (nups_shard_table*)calloc(1, sizeof(nups_shard_table));
    if (!t) return NUPS_ENOMEM;
    t->num_keys = num_keys;
    t->value_len = value_len;
    t->n_shards = n_shards;
    t->my_shard = my_shard;
    t->keys_per_shard = (num_keys + n_shards - 1) / n_shards;
    const size_t bytes = (size_t)t->keys_per_shard * value_len * sizeof(float);
    cudaError_t e = cudaGetDevice(&t->device);
    if (e == cudaSuccess) e = cudaMalloc((void**)&t->local, bytes);
    if (e == cudaSuccess) e = cudaMemset(t->local, 0, bytes);
    if (e == cudaSuccess) e = cudaMalloc((void**)&t->base_d, NUPS_MAX_SHARDS * sizeof(float*));
    if (e == cudaSuccess) e = cudaMalloc((void**)&t->status_d, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(t->status_d, 0, sizeof(int));
    if (e != cudaSuccess) {
        const bool oom = e == cudaErrorMemoryAllocation;
        cudaGetLastError();
        cudaFree(t->local); cudaFree(t->base_d); cudaFree(t->status_d);
        free(t);
        return oom ? NUPS_ENOMEM : NUPS_ECUDA;
    }
    t->base_h[my_shard] = t->local;
    t->bases_changed = true;
    *out = t;
    return NUPS_OK;
}

extern "C" void nups_shard_table_destroy(nups_shard_table* t)
{
    if (!t) return;
    for (uint32_t j = 0; j < NUPS_MAX_SHARDS; ++j)
        if (t->ipc_opened[j]) cudaIpcCloseMemHandle(t->ipc_opened[j]);
    cudaFree(t->local);
    cudaFree(t->base_d);
    cudaFree(t->status_d);
    cudaGetLastError();
    free(t);
}

extern "C" const char* nups_shard_last_error(const nups_shard_table* t) { return t ? t->err : ""; }

extern "C" nups_status nups_shard_table_local(nups_shard_table* t, void** h_ptr_out, uint64_t* h_bytes_out)
{
    if (!t || !h_ptr_out || !h_bytes_out) return NUPS_EINVAL;
    *h_ptr_out = t->local;
    *h_bytes_out = (uint64_t)t->keys_per_shard * t->value_len * sizeof(float);
    return NUPS_OK;
}

static_assert(sizeof(cudaIpcMemHandle_t) == NUPS_SHARD_HANDLE_BYTES, "the exported handle is a cudaIpcMemHandle_t");

extern "C" nups_status nups_shard_table_export(nups_shard_table* t, unsigned char* h_handle_out)
{
    if (!t || !h_handle_out) return NUPS_EINVAL;
    cudaIpcMemHandle_t h;
    SCK(t, cudaIpcGetMemHandle(&h, t->local));
    memcpy(h_handle_out, &h, sizeof(h));
    return NUPS_OK;
}

extern "C" nups_status nups_shard_table_attach(nups_shard_table* t, uint32_t shard, void* d_first_row)
{
    if (!t || shard >= t->n_shards || shard == t->my_shard || !d_first_row || ((uintptr_t)d_first_row & 15)) return NUPS_EINVAL;
    if (t->ipc_opened[shard]) { cudaIpcCloseMemHandle(t->ipc_opened[shard]); t->ipc_opened[shard] = nullptr; }
    t->base_h[shard] = (float*)d_first_row;
    t->bases_changed = true;
    return NUPS_OK;
}

extern "C" nups_status nups_shard_table_attach_ipc(nups_shard_table* t, uint32_t shard, const unsigned char* h_handle)
{
    if (!t || shard >= t->n_shards || shard == t->my_shard || !h_handle) return NUPS_EINVAL;
    cudaIpcMemHandle_t h;
    memcpy(&h, h_handle, sizeof(h));
    void* p = nullptr;
    SCK(t, cudaIpcOpenMemHandle(&p, h, cudaIpcMemLazyEnablePeerAccess));
    if (t->ipc_opened[shard]) cudaIpcCloseMemHandle(t->ipc_opened[shard]);
    t->ipc_opened[shard] = p;
    t->base_h[shard] = (float*)p;
    t->bases_changed = true;
    return NUPS_OK;
}

extern "C" nups_status nups_shard_table_copy(nups_shard_table* t, void* d_rows, int to_table, void* stream)
{
    if (!t || !d_rows) return NUPS_EINVAL;
    const size_t bytes = (size_t)t->keys_per_shard * t->value_len * sizeof(float);
    SCK(t, cudaMemcpyAsync(to_table ? (void*)t->local : d_rows, to_table ? d_rows : (void*)t->local, bytes,
                           cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return NUPS_OK;
}

// every shard attached?  then make sure the device sees the current addresses
static nups_status shard_ready(nups_shard_table* t, cudaStream_t st)
{
    for (uint32_t j = 0; j < t->n_shards; ++j)
        if (!t->base_h[j]) return NUPS_ESTATE;
    if (t->bases_changed) {
        // the copy reads base_h when it is issued (pageable memory), so a later attach cannot reach an earlier call
        SCK(t, cudaMemcpyAsync(t->base_d, t->base_h, NUPS_MAX_SHARDS * sizeof(float*), cudaMemcpyHostToDevice, st));
        SCK(t, cudaStreamSynchronize(st));
        t->bases_changed = false;
    }
    return NUPS_OK;
}

struct ShardView {
    const unsigned long long* base;   // [n_shards] address of the first row of every shard
    uint64_t num_keys;
    uint32_t keys_per_shard, L4;
    int* status;
};

constexpr int SHARD_UNROLL = 4;
constexpr unsigned long long SHARD_NO_ROW = 0ull;         // a null address: the row is skipped

// address of a key's row (as an integer, to pass it between lanes), or SHARD_NO_ROW for a key out of range
__device__ __forceinline__ unsigned long long shard_row(const ShardView& sv, uint32_t key, bool in)
{
    if (!in) return SHARD_NO_ROW;
    if (key >= sv.num_keys) { atomicCAS(sv.status, 0, NUPS_EKEY); return SHARD_NO_ROW; }
    const uint32_t owner = key / sv.keys_per_shard, local = key - owner * sv.keys_per_shard;
    return __ldg(sv.base + owner) + (unsigned long long)local * sv.L4 * 16;
}

// pull: a warp walks windows of 32 keys; every lane turns one key into the address of its row in the owner's memory;
// the warp then copies the rows SHARD_UNROLL at a time with 128-bit loads (from local HBM or over NVLink, the kernel
// does not care which) and streaming stores
__global__ void __launch_bounds__(256, 4)
shard_gather_kernel(ShardView sv, const uint32_t* __restrict__ keys, uint64_t n, float4* __restrict__ out)
{
    grid_dependency_wait();
    const unsigned lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t stride = (((uint64_t)gridDim.x * blockDim.x) >> 5) * 32;
    const uint32_t L4 = sv.L4;
    uint64_t base = warp * 32;
    uint32_t key_next = base + lane < n ? __ldg(keys + base + lane) : 0u;
    for (; base < n; base += stride) {
        const uint32_t key = key_next;
        key_next = base + stride + lane < n ? __ldg(keys + base + stride + lane) : 0u;
        const unsigned long long src = shard_row(sv, key, base + lane < n);
        const int rows = (int)min((uint64_t)32, n - base);
        for (int r = 0; r < rows; r += SHARD_UNROLL) {
            unsigned long long so[SHARD_UNROLL];
#pragma unroll
            for (int u = 0; u < SHARD_UNROLL; ++u) so[u] = __shfl_sync(0xFFFFFFFFu, src, min(r + u, 31));
            for (uint32_t c = lane; c < L4; c += 32) {
                float4 a[SHARD_UNROLL];
#pragma unroll
                for (int u = 0; u < SHARD_UNROLL; ++u) {
                    a[u] = make_float4(0.f, 0.f, 0.f, 0.f);                       // a skipped row is zero-filled
                    if (r + u < rows && so[u] != SHARD_NO_ROW) a[u] = ld_stream_v4(reinterpret_cast<const float4*>(so[u]) + c);
                }
#pragma unroll
                for (int u = 0; u < SHARD_UNROLL; ++u)
                    if (r + u < rows) st_stream_v4(out + (base + r + u) * L4 + c, a[u]);
            }
        }
    }
}

// push: the same walk; every row of the caller's updates is added to its key's row where that row lives, by 128-bit
// floating-point reductions (to local HBM or to a peer's over NVLink).  Rows of one window that go to the same key are
// summed in registers first, so that a frequent key takes one reduction per window rather than one per row; keys hot
// enough to need more than that belong, replicated, in the per-GPU store.
__global__ void __launch_bounds__(256, 4)
shard_push_kernel(ShardView sv, const uint32_t* __restrict__ keys, uint64_t n, const float4* __restrict__ delta)
{
    grid_dependency_wait();
    const unsigned lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t stride = (((uint64_t)gridDim.x * blockDim.x) >> 5) * 32;
    const uint32_t L4 = sv.L4;
    uint64_t base = warp * 32;
    uint32_t key_next = base + lane < n ? __ldg(keys + base + lane) : 0u;
    for (; base < n; base += stride) {
        const uint32_t key = key_next;
        key_next = base + stride + lane < n ? __ldg(keys + base + stride + lane) : 0u;
        const unsigned long long dst = shard_row(sv, key, base + lane < n);
        const bool valid = dst != SHARD_NO_ROW;
        // lanes with the same destination; a skipped row gets a value of its own (an odd number: no row address is odd)
        const unsigned grp = __match_any_sync(0xFFFFFFFFu, valid ? dst : (unsigned long long)(2 * lane + 1));
        const bool leader = valid && lane == (unsigned)(__ffs(grp) - 1);
        unsigned singles = __ballot_sync(0xFFFFFFFFu, leader && __popc(grp) == 1);
        unsigned multis = __ballot_sync(0xFFFFFFFFu, leader && __popc(grp) > 1);
        while (singles) {                                          // rows alone in their window: SHARD_UNROLL at a time
            int src[SHARD_UNROLL];
            unsigned long long to[SHARD_UNROLL];
#pragma unroll
            for (int u = 0; u < SHARD_UNROLL; ++u) {
                src[u] = singles ? __ffs(singles) - 1 : -1;
                singles &= singles - 1;
                to[u] = __shfl_sync(0xFFFFFFFFu, dst, src[u] < 0 ? 0 : src[u]);
            }
            for (uint32_t c = lane; c < L4; c += 32) {
                float4 a[SHARD_UNROLL];
#pragma unroll
                for (int u = 0; u < SHARD_UNROLL; ++u)
                    if (src[u] >= 0) a[u] = ld_stream_v4(delta + (base + src[u]) * L4 + c);
#pragma unroll
                for (int u = 0; u < SHARD_UNROLL; ++u)
                    if (src[u] >= 0) red_add_v4(reinterpret_cast<float*>(to[u]) + 4 * c, a[u]);
            }
        }
        while (multis) {                                           // a key hit several times: sum its rows, one reduction
            const int ld = __ffs(multis) - 1;
            multis &= multis - 1;
            const unsigned members = __shfl_sync(0xFFFFFFFFu, grp, ld);
            const unsigned long long to = __shfl_sync(0xFFFFFFFFu, dst, ld);
            for (uint32_t c = lane; c < L4; c += 32) {
                float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
                unsigned mm = members;
                while (mm) {
                    int m[SHARD_UNROLL];
                    float4 x[SHARD_UNROLL];
#pragma unroll
                    for (int u = 0; u < SHARD_UNROLL; ++u) {
                        m[u] = mm ? __ffs(mm) - 1 : -1;
                        mm &= mm - 1;
                    }
#pragma unroll
                    for (int u = 0; u < SHARD_UNROLL; ++u)
                        if (m[u] >= 0) x[u] = ld_stream_v4(delta + (base + m[u]) * L4 + c);
#pragma unroll
                    for (int u = 0; u < SHARD_UNROLL; ++u)
                        if (m[u] >= 0) sum = add4(sum, x[u]);
                }
                red_add_v4(reinterpret_cast<float*>(to) + 4 * c, sum);
            }
        }
    }
}

static ShardView shard_view(const nups_shard_table* t)
{
    ShardView sv;
    sv.base = reinterpret_cast<const unsigned long long*>(t->base_d);
    sv.num_keys = t->num_keys;
    sv.keys_per_shard = (uint32_t)t->keys_per_shard;
    sv.L4 = t->value_len / 4;
    sv.status = t->status_d;
    return sv;
}

static unsigned shard_grid(uint64_t n)
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 148;
    return grid_for(n, 256, (unsigned)sms * 4);              // resident at once, grid-stride
}

extern "C" nups_status nups_shard_pull(nups_shard_table* t, const uint32_t* d_keys, uint64_t n, void* d_out, void* stream)
{
    if (!t || (n && (!d_keys || !d_out)) || n >= (1ull << 32) || ((uintptr_t)d_out & 15)) return NUPS_EINVAL;
    if (n == 0) return NUPS_OK;
    cudaStream_t st = (cudaStream_t)stream;
    nups_status rc = shard_ready(t, st);
    if (rc != NUPS_OK) return rc;
    SCK(t, nups_launch_dependent(shard_gather_kernel, shard_grid(n), 256, 0, st, shard_view(t), d_keys, n, (float4*)d_out));
    return NUPS_OK;
}

extern "C" nups_status nups_shard_push(nups_shard_table* t, const uint32_t* d_keys, uint64_t n, const void* d_delta, void* stream)
{
    if (!t || (n && (!d_keys || !d_delta)) || n >= (1ull << 32) || ((uintptr_t)d_delta & 15)) return NUPS_EINVAL;
    if (n == 0) return NUPS_OK;
    cudaStream_t st = (cudaStream_t)stream;
    nups_status rc = shard_ready(t, st);
    if (rc != NUPS_OK) return rc;
    SCK(t, nups_launch_dependent(shard_push_kernel, shard_grid(n), 256, 0, st, shard_view(t), d_keys, n, (const float4*)d_delta));
    return NUPS_OK;
}

extern "C" nups_status nups_shard_status_check(nups_shard_table* t, void* stream)
{
    if (!t) return NUPS_EINVAL;
    int h = 0;
    SCK(t, cudaMemcpyAsync(&h, t->status_d, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    SCK(t, cudaStreamSynchronize((cudaStream_t)stream));
    if (h != 0) {
        SCK(t, cudaMemsetAsync(t->status_d, 0, sizeof(int), (cudaStream_t)stream));
        return (nups_status)h;
    }
    return NUPS_OK;
}

// ---------------------------------------------------------------------------------------------
// Merging a replicated store across GPUs (Section 3.2: replicas are synchronised by an all-reduce of their accumulated
// updates).  Every GPU keeps a whole nups_store of the keys that are replicated across GPUs (a small one: the hot keys)
// and updates it on its own.  `snap` is the table as all GPUs last agreed on it.  A merge is three steps: every GPU
// exports own = table - snap (after merging its own workers' replicas into the table); the caller adds the exported
// buffers up over all GPUs (one all-reduce); every GPU applies table += total - own and snap += total.  Afterwards all
// tables are the agreed values plus whatever each GPU added since its export, which the next merge carries over:
// nothing that arrives between export and apply is lost, and the additions to the table are reductions, so pushes may
// run beside them.
// ---------------------------------------------------------------------------------------------
template <class T>
__global__ void merge_export_kernel(const T* __restrict__ table, const T* __restrict__ snap, T* __restrict__ own, uint64_t n)
{
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x)
        own[i] = table[i] - snap[i];
}

template <class T>
__global__ void merge_apply_kernel(T* table, T* __restrict__ snap, const T* __restrict__ total, const T* __restrict__ own,
                                   uint64_t n)
{
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
        const T t = total[i], others = t - own[i];
        if (others != T(0)) atomicAdd(table + i, others);
        snap[i] += t;
    }
}

static bool merge_args_ok(const nups_store* s, int which)
{
    return s && (which == 0 || which == 1) && (which == 0 || s->acc);
}

extern "C" nups_status nups_merge_mark(nups_store* s, int which, void* stream)
{
    if (!merge_args_ok(s, which)) return NUPS_EINVAL;
    const size_t bytes = (size_t)s->num_keys * s->L * sizeof(float);
    if (!s->merge_snap[which]) {
        nups_status rc = nups_dev_alloc(s, (void**)&s->merge_snap[which], bytes);
        if (rc != NUPS_OK) return rc;
    }
    nups_status rc = nups_sync_internal(s, (cudaStream_t)stream);           // the workers' replicas belong to the table
    if (rc != NUPS_OK) return rc;
    CK(cudaMemcpyAsync(s->merge_snap[which], which ? s->acc : s->val, bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return NUPS_OK;
}

extern "C" nups_status nups_merge_export(nups_store* s, int which, void* d_own_out, void* stream)
{
    if (!merge_args_ok(s, which) || !d_own_out) return NUPS_EINVAL;
    if (!s->merge_snap[which]) return NUPS_ESTATE;
    cudaStream_t st = (cudaStream_t)stream;
    nups_status rc = nups_sync_internal(s, st);
    if (rc != NUPS_OK) return rc;
    const uint64_t words = (uint64_t)s->num_keys * s->L;
    const void* table = which ? s->acc : s->val;
    if (s->vb == 8)
        merge_export_kernel<double><<<grid_for(words / 2, 256, (unsigned)s->sm_count * 8), 256, 0, st>>>(
            (const double*)table, (const double*)s->merge_snap[which], (double*)d_own_out, words / 2);
    else
        merge_export_kernel<float><<<grid_for(words, 256, (unsigned)s->sm_count * 8), 256, 0, st>>>(
            (const float*)table, s->merge_snap[which], (float*)d_own_out, words);
    LAUNCH_CHECK(s);
    return NUPS_OK;
}

extern "C" nups_status nups_merge_apply(nups_store* s, int which, const void* d_total, const void* d_own, void* stream)
{
    if (!merge_args_ok(s, which) || !d_total || !d_own) return NUPS_EINVAL;
    if (!s->merge_snap[which]) return NUPS_ESTATE;
    cudaStream_t st = (cudaStream_t)stream;
    const uint64_t words = (uint64_t)s->num_keys * s->L;
    void* table = which ? s->acc : s->val;
    if (s->vb == 8)
        merge_apply_kernel<double><<<grid_for(words / 2, 256, (unsigned)s->sm_count * 8), 256, 0, st>>>(
            (double*)table, (double*)s->merge_snap[which], (const double*)d_total, (const double*)d_own, words / 2);
    else
        merge_apply_kernel<float><<<grid_for(words, 256, (unsigned)s->sm_count * 8), 256, 0, st>>>(
            (float*)table, s->merge_snap[which], (const float*)d_total, (const float*)d_own, words);
    LAUNCH_CHECK(s);
    return NUPS_OK;
}
