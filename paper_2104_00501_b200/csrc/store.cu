// Key store, direct access (pull / push), replica merge, access counting, hot-set selection and
// per-key management.  NuPS Sections 3.1, 3.2, 5.1.
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "nups_internal.cuh"

thread_local char g_nups_cuda_err[256] = "";

nups_status nups_cuda_fail(cudaError_t e, const char* what)
{
    snprintf(g_nups_cuda_err, sizeof(g_nups_cuda_err), "%s: %s", what, cudaGetErrorString(e));
    return NUPS_ECUDA;
}

extern "C" const char* nups_last_cuda_error(void) { return g_nups_cuda_err; }

extern "C" const char* nups_strerror(nups_status st)
{
    switch (st) {
        case NUPS_OK: return "ok";
        case NUPS_EINVAL: return "invalid argument";
        case NUPS_ENOMEM: return "out of memory or table full";
        case NUPS_ECUDA: return "CUDA runtime error";
        case NUPS_EKEY: return "key out of range seen on the device";
        case NUPS_ESTATE: return "call not valid in the current state";
        case NUPS_ETIMEOUT: return "bounded device-side wait gave up";
        default: return "unknown status";
    }
}

View nups_view(const nups_store* s)
{
    View v;
    v.val = s->val; v.acc = s->acc; v.dval = s->dval; v.dacc = s->dacc;
    v.hot_bits = s->hot_bits; v.slot_of = s->slot_of; v.dirty = s->dirty;
    v.cnt = s->cnt; v.own = s->own; v.epoch_tag = s->epoch << 8; v.st = s->st; v.loss_partial = s->loss_partial;
    v.num_keys = s->num_keys; v.Hcap = s->Hcap; v.H = (uint32_t)s->H; v.L4 = s->L / 4; v.R = s->R;
    v.count = s->cfg.count_accesses;
    v.merge_mean = s->cfg.merge_mean;
    v.f64 = s->vb == 8;
    v.clip_factor = s->cfg.clip_factor;
    return v;
}

nups_status nups_dev_alloc(nups_store* s, void** p, size_t bytes)
{
    *p = nullptr;
    if (bytes == 0) return NUPS_OK;
    if (s->dev_cap && (bytes > s->dev_cap || s->dev_bytes > s->dev_cap - bytes)) return NUPS_ENOMEM;   // the store's own limit
    if (cudaMalloc(p, bytes) != cudaSuccess) {
        cudaGetLastError();
        *p = nullptr;
        return NUPS_ENOMEM;
    }
    s->dev_bytes += bytes;
    return NUPS_OK;
}

void nups_dev_free(nups_store* s, void* p, size_t bytes)
{
    if (!p) return;
    cudaFree(p);                                   // waits for work that may still use it
    s->dev_bytes -= bytes < s->dev_bytes ? bytes : s->dev_bytes;
}

nups_status nups_scratch(nups_store* s, size_t bytes, char** out)
{
    if (bytes > s->scratch_bytes) {
        size_t want = bytes + bytes / 4 + (1u << 20);
        // the limit is judged with the old buffer already handed back; on refusal the old buffer stays
        if (s->dev_cap && (want > s->dev_cap || s->dev_bytes - s->scratch_bytes > s->dev_cap - want)) return NUPS_ENOMEM;
        nups_dev_free(s, s->scratch, s->scratch_bytes);
        s->scratch = nullptr; s->scratch_bytes = 0;
        nups_status rc = nups_dev_alloc(s, (void**)&s->scratch, want);
        if (rc != NUPS_OK) return rc;
        s->scratch_bytes = want;
    }
    *out = s->scratch;
    return NUPS_OK;
}

// Calls that move keys are numbered; the number is stored above the owner in every word such a call
// writes.  When the 24 bits run out, the numbers in the table are cleared and counting restarts.
__global__ void own_clear_epoch_kernel(uint32_t* own, uint64_t n)
{
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (; i < n; i += stride) own[i] &= 0xFFu;
}

nups_status nups_new_epoch(nups_store* s, cudaStream_t st)
{
    if (!s->own) return NUPS_OK;
    if (s->epoch >= 0xFFFFFFu) {
        own_clear_epoch_kernel<<<grid_for(s->num_keys, 256, 8192), 256, 0, st>>>(s->own, s->num_keys);
        LAUNCH_CHECK(s);
        s->epoch = 0;
    }
    s->epoch++;
    return NUPS_OK;
}

static inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// ---------------------------------------------------------------------------------------------
// optional event pairs around the main kernels (benchmark aid)
// ---------------------------------------------------------------------------------------------
static void timing_fold(nups_store* s)
{
    for (uint32_t i = 0; i < s->ev_n; ++i) {
        float ms = 0.f;
        const int kind = s->ev_kind[i];
        if (cudaEventSynchronize(s->ev[2 * i + 1]) == cudaSuccess &&
            cudaEventElapsedTime(&ms, s->ev[2 * i], s->ev[2 * i + 1]) == cudaSuccess)
            s->ev_ms[kind] += ms;
        s->ev_launches[kind]++;
    }
    s->ev_n = 0;
    cudaGetLastError();
}
void nups_time_begin(nups_store* s, cudaStream_t st, int kind)
{
    if (!s->timing) return;
    if (s->ev_n == NUPS_MAX_TIMED) timing_fold(s);
    s->ev_kind[s->ev_n] = (unsigned char)kind;
    cudaEventRecord(s->ev[2 * s->ev_n], st);
}
void nups_time_end(nups_store* s, cudaStream_t st)
{
    if (!s->timing) return;
    cudaEventRecord(s->ev[2 * s->ev_n + 1], st);
    s->ev_n++;
}
static void timing_clear(nups_store* s)
{
    for (int k = 0; k < NUPS_TIMED_KINDS; ++k) { s->ev_ms[k] = 0; s->ev_launches[k] = 0; }
}
extern "C" nups_status nups_kernel_timing(nups_store* s, int enable)
{
    if (!s) return NUPS_EINVAL;
    if (enable && !s->ev) {
        s->ev = (cudaEvent_t*)calloc(2 * NUPS_MAX_TIMED, sizeof(cudaEvent_t));
        s->ev_kind = (unsigned char*)calloc(NUPS_MAX_TIMED, 1);
        if (!s->ev || !s->ev_kind) return NUPS_ENOMEM;
        for (int i = 0; i < 2 * NUPS_MAX_TIMED; ++i) CK(cudaEventCreate(&s->ev[i]));
    }
    s->timing = enable ? 1 : 0;       // what was recorded stays until it is queried: switching costs no synchronisation
    return NUPS_OK;
}
extern "C" nups_status nups_kernel_times(nups_store* s, double* h_ms_out, uint64_t* h_launches_out, void* stream)
{
    if (!s || !h_ms_out || !h_launches_out) return NUPS_EINVAL;
    CK(cudaStreamSynchronize((cudaStream_t)stream));
    if (s->ev) timing_fold(s);
    for (int k = 0; k < NUPS_TIMED_KINDS; ++k) { h_ms_out[k] = s->ev_ms[k]; h_launches_out[k] = s->ev_launches[k]; }
    timing_clear(s);
    return NUPS_OK;
}
extern "C" nups_status nups_kernel_time(nups_store* s, double* h_ms_out, uint64_t* h_launches_out, void* stream)
{
    if (!s || !h_ms_out || !h_launches_out) return NUPS_EINVAL;
    double ms[NUPS_TIMED_KINDS];
    uint64_t n[NUPS_TIMED_KINDS];
    nups_status rc = nups_kernel_times(s, ms, n, stream);
    if (rc != NUPS_OK) return rc;
    *h_ms_out = 0; *h_launches_out = 0;
    for (int k = 0; k < NUPS_TIMED_KINDS; ++k) { *h_ms_out += ms[k]; *h_launches_out += n[k]; }
    return NUPS_OK;
}

// ---------------------------------------------------------------------------------------------
// create / destroy
// ---------------------------------------------------------------------------------------------
__global__ void fill_i32(int* p, uint64_t n, int value)
{
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (; i < n; i += stride) p[i] = value;
}

extern "C" nups_status nups_create(uint64_t num_keys, uint32_t value_len, const nups_config* cfg, nups_store** out)
{
    if (!out) return NUPS_EINVAL;
    *out = nullptr;
    if (num_keys == 0 || num_keys > 0xFFFFFFFFull || value_len == 0) return NUPS_EINVAL;
    nups_config c;
    memset(&c, 0, sizeof(c));
    if (cfg) c = *cfg;
    if (c.value_bytes == 0) c.value_bytes = 4;
    if (c.value_bytes != 4 && c.value_bytes != 8) return NUPS_EINVAL;
    if (((uint64_t)value_len * c.value_bytes) & 15) return NUPS_EINVAL;       // rows are multiples of 16 bytes
    if (c.value_bytes == 8 && (c.clip_factor > 0.f || c.sync_period_us)) return NUPS_EINVAL;
    if ((uint64_t)value_len * (c.value_bytes / 4) > 0xFFFFFFFFull) return NUPS_EINVAL;
    const uint32_t units = value_len * (c.value_bytes / 4);                     // row length in 4-byte units
    if (c.workers == 0) c.workers = 8;
    if (c.workers > 254) return NUPS_EINVAL;
    if (c.sync_period_us && c.deterministic) return NUPS_EINVAL;
    if (!(c.clip_factor >= 0.f)) return NUPS_EINVAL;
    if (c.merge_mean > 1 || (c.merge_mean && c.sync_period_us)) return NUPS_EINVAL;
    if (c.first_epoch > 0xFFFFFFu) return NUPS_EINVAL;
    // what the store holds from the start: tables, technique bitmap, slot map, counts, ownership words, status, loss words
    const size_t table_bytes = (size_t)num_keys * units * sizeof(float);
    const size_t bits_bytes = ((num_keys + 31) / 32) * 4, loss_bytes = 4 * NUPS_MAX_STEP_BLOCKS * sizeof(double);
    const size_t need = table_bytes * (c.with_adagrad ? 2 : 1) + bits_bytes + num_keys * 4 + num_keys * 8 +
                        (c.track_ownership ? num_keys * 4 : 0) + sizeof(DevStat) + loss_bytes;
    const size_t cap = (size_t)c.max_device_mib << 20;
    if (cap && need > cap) return NUPS_ENOMEM;              // the store's own limit, judged before the device is touched
    int dev = 0, count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || count == 0) {
        snprintf(g_nups_cuda_err, sizeof(g_nups_cuda_err), "no CUDA device");
        cudaGetLastError();
        return NUPS_ECUDA;
    }
    CK(cudaGetDevice(&dev));
    nups_store* s = (nups_store*)calloc(1, sizeof(nups_store));
    if (!s) return NUPS_ENOMEM;
    s->num_keys = num_keys; s->L = units; s->value_len = value_len; s->vb = c.value_bytes; s->R = c.workers; s->cfg = c;
    s->device = dev;
    s->dev_cap = cap;
    s->epoch = c.first_epoch;
    s->ahead_dist = -1;
    cudaDeviceGetAttribute(&s->sm_count, cudaDevAttrMultiProcessorCount, dev);
    cudaDeviceGetAttribute(&s->max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    bool ok = nups_dev_alloc(s, (void**)&s->val, table_bytes) == NUPS_OK;
    if (ok && c.with_adagrad) ok = nups_dev_alloc(s, (void**)&s->acc, table_bytes) == NUPS_OK;
    ok = ok && nups_dev_alloc(s, (void**)&s->hot_bits, bits_bytes) == NUPS_OK;
    ok = ok && nups_dev_alloc(s, (void**)&s->slot_of, num_keys * 4) == NUPS_OK;
    ok = ok && nups_dev_alloc(s, (void**)&s->cnt, num_keys * 8) == NUPS_OK;
    ok = ok && nups_dev_alloc(s, (void**)&s->st, sizeof(DevStat)) == NUPS_OK;
    ok = ok && nups_dev_alloc(s, (void**)&s->loss_partial, loss_bytes) == NUPS_OK;
    if (ok && c.track_ownership) ok = nups_dev_alloc(s, (void**)&s->own, num_keys * 4) == NUPS_OK;
    if (!ok) {
        cudaGetLastError();
        nups_destroy(s);
        return NUPS_ENOMEM;
    }
    cudaMemset(s->val, 0, table_bytes);
    if (s->acc) cudaMemset(s->acc, 0, table_bytes);
    cudaMemset(s->hot_bits, 0, ((num_keys + 31) / 32) * 4);
    cudaMemset(s->cnt, 0, num_keys * 8);
    cudaMemset(s->st, 0, sizeof(DevStat));
    cudaMemset(s->loss_partial, 0, 4 * NUPS_MAX_STEP_BLOCKS * sizeof(double));
    fill_i32<<<grid_for(num_keys, 256, 4096), 256>>>(s->slot_of, num_keys, -1);
    if (s->own) {
        fill_i32<<<grid_for(num_keys, 256, 4096), 256>>>((int*)s->own, num_keys, NUPS_OWNER_DEFAULT);
    }
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        nups_destroy(s);
        return nups_cuda_fail(e, "nups_create");
    }
    if (c.sync_period_us) {
        nups_status rc = nups_background_start(s, c.sync_period_us);
        if (rc != NUPS_OK) {
            nups_destroy(s);
            return rc;
        }
    }
    *out = s;
    return NUPS_OK;
}

extern "C" nups_status nups_destroy(nups_store* s)
{
    if (!s) return NUPS_OK;
    nups_background_stop(s);
    cudaDeviceSynchronize();
    if (s->side) { cudaStreamDestroy(s->side); cudaEventDestroy(s->side_fork); cudaEventDestroy(s->side_join); }
    for (int i = 0; i < NUPS_MAX_HANDLES; ++i) cudaFree(s->handle[i].buf);
    for (int i = 0; i < NUPS_MAX_DISTS; ++i) { cudaFree(s->dist[i].table); cudaFree(s->dist[i].off); }
    cudaFree(s->val); cudaFree(s->acc); cudaFree(s->hot_bits); cudaFree(s->slot_of); cudaFree(s->hot_keys);
    cudaFree(s->dval); cudaFree(s->dacc); cudaFree(s->dirty); cudaFree(s->cnt); cudaFree(s->own);
    cudaFree(s->st); cudaFree(s->loss_partial); cudaFree(s->scratch); cudaFree(s->negs_buf);
    cudaFree(s->merge_snap[0]); cudaFree(s->merge_snap[1]);
    if (s->ev) {
        for (int i = 0; i < 2 * NUPS_MAX_TIMED; ++i) cudaEventDestroy(s->ev[i]);
        free(s->ev);
        free(s->ev_kind);
    }
    cudaGetLastError();
    free(s);
    return NUPS_OK;
}

extern "C" nups_status nups_table_ptr(nups_store* s, int which, void** ptr, uint64_t* stride)
{
    if (!s || !ptr || (which != 0 && which != 1)) return NUPS_EINVAL;
    if (which == 1 && !s->acc) return NUPS_EINVAL;
    *ptr = which ? s->acc : s->val;
    if (stride) *stride = s->value_len;
    return NUPS_OK;
}

extern "C" nups_status nups_table_copy(nups_store* s, int which, void* d_buf, int to_store, void* stream)
{
    if (!s || !d_buf || (which != 0 && which != 1) || (which == 1 && !s->acc)) return NUPS_EINVAL;
    void* t = which ? s->acc : s->val;
    size_t bytes = (size_t)s->num_keys * s->L * sizeof(float);
    CK(cudaMemcpyAsync(to_store ? t : d_buf, to_store ? d_buf : t, bytes, cudaMemcpyDeviceToDevice,
                       (cudaStream_t)stream));
    return NUPS_OK;
}

__global__ void init_uniform_kernel(float4* t, uint64_t total4, uint64_t seed, uint32_t which, float unit)
{
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (; i < total4; i += stride) {
        uint32_t x[4];
        philox_at(seed, i, which, 3, 0, x);
        float4 r;
        r.x = __fmul_rn((float)((int)(x[0] >> 8) - 8388608), unit);
        r.y = __fmul_rn((float)((int)(x[1] >> 8) - 8388608), unit);
        r.z = __fmul_rn((float)((int)(x[2] >> 8) - 8388608), unit);
        r.w = __fmul_rn((float)((int)(x[3] >> 8) - 8388608), unit);
        t[i] = r;
    }
}

// the same values (each exactly representable in fp32) into a table of doubles
__global__ void init_uniform_f64_kernel(double* t, uint64_t total4, uint64_t seed, uint32_t which, float unit)
{
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (; i < total4; i += stride) {
        uint32_t x[4];
        philox_at(seed, i, which, 3, 0, x);
#pragma unroll
        for (int k = 0; k < 4; ++k) t[4 * i + k] = (double)__fmul_rn((float)((int)(x[k] >> 8) - 8388608), unit);
    }
}

extern "C" nups_status nups_init_uniform(nups_store* s, int which, uint64_t seed, float scale, void* stream)
{
    if (!s || (which != 0 && which != 1) || (which == 1 && !s->acc)) return NUPS_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    const uint64_t values = s->num_keys * (uint64_t)s->value_len;
    if (values & 3) return NUPS_EINVAL;                       // the generator makes four values at a time
    const uint64_t total4 = values / 4;
    float unit = scale * (1.0f / 8388608.0f);
    const unsigned grid = grid_for(total4, 256, (unsigned)s->sm_count * 16);
    if (s->vb == 8)
        init_uniform_f64_kernel<<<grid, 256, 0, st>>>((double*)(which ? s->acc : s->val), total4, seed, (uint32_t)which, unit);
    else
        init_uniform_kernel<<<grid, 256, 0, st>>>((float4*)(which ? s->acc : s->val), total4, seed, (uint32_t)which, unit);
    LAUNCH_CHECK(s);
    return NUPS_OK;
}

// ---------------------------------------------------------------------------------------------
// pull: row gather.  One warp walks windows of 32 keys; each lane fetches one key of the window and
// turns it into the offset of its row (and of the worker's pending replica row, if the key is
// replicated); the warp then copies the rows four at a time with 128-bit loads and streaming
// stores.  TWO = also copy the matching rows of a second table.
// ---------------------------------------------------------------------------------------------
constexpr int GATHER_UNROLL = 4;
constexpr unsigned long long NO_ROW = ~0ull;

struct TablePair {
    const float4* table;   // stored rows
    const float4* slab;    // pending replica updates [R][Hcap][L]
    float4* out;           // [n][L]
};

template <bool HOT, bool TWO, bool F64>
__global__ void __launch_bounds__(256, 4)
gather_kernel(View v, const uint32_t* __restrict__ keys, uint64_t n, TablePair A, TablePair B, int map,
              uint64_t map_base, uint64_t map_total, int do_count, uint32_t* __restrict__ keys_copy)
{
    grid_dependency_wait();
    const unsigned lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t nwarps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    const uint32_t L4 = v.L4;
    // Lookups run ahead of the copies: while window w is copied, the key of window w + 2 and the
    // hot-bit word of window w + 1 are already on their way.
    const uint64_t stride = nwarps * 32;
    uint64_t base = warp * 32;
    uint32_t key_a = base + lane < n ? __ldg(keys + base + lane) : 0u;                         // window w
    uint32_t key_b = base + stride + lane < n ? __ldg(keys + base + stride + lane) : 0u;       // window w + 1
    uint32_t bits_a = (HOT && key_a < v.num_keys) ? __ldg(v.hot_bits + (key_a >> 5)) : 0u;
    for (; base < n; base += stride) {
        const uint64_t i = base + lane;
        const bool in = i < n;
        const uint32_t key = key_a;
        const uint32_t bits = bits_a;
        key_a = key_b;
        bits_a = (HOT && key_a < v.num_keys) ? __ldg(v.hot_bits + (key_a >> 5)) : 0u;
        key_b = base + 2 * stride + lane < n ? __ldg(keys + base + 2 * stride + lane) : 0u;
        const bool valid = in && key < v.num_keys;
        if (in && !valid) flag_bad_key(v);
        if (keys_copy && in) keys_copy[i] = key;                   // PullSample hands the keys out as well
        unsigned long long src = valid ? (unsigned long long)key * L4 : NO_ROW;   // NO_ROW: zero-filled output
        unsigned long long pend = NO_ROW;
        if (HOT && valid && ((bits >> (key & 31)) & 1u)) {
            const uint32_t slot = (uint32_t)__ldg(v.slot_of + key);
            const uint64_t idx = map_base + i;
            const uint32_t q = map == 0 ? worker_of_item(idx, map_total, v.R) : chunk_of_pos(idx, map_total, v.R);
            pend = ((unsigned long long)q * v.Hcap + slot) * L4;
        }
        if (do_count && v.count) {
            if (valid) atomicAdd(v.cnt + key, 1ull);
            unsigned hot_m = __ballot_sync(0xFFFFFFFFu, valid && pend != NO_ROW);
            unsigned cold_m = __ballot_sync(0xFFFFFFFFu, valid && pend == NO_ROW);
            if (lane == 0) {
                if (hot_m) atomicAdd(&v.st->hot_hits, (unsigned long long)__popc(hot_m));
                if (cold_m) atomicAdd(&v.st->cold_hits, (unsigned long long)__popc(cold_m));
            }
        }
        const int rows = (int)min((uint64_t)32, n - base);
        for (int r = 0; r < rows; r += GATHER_UNROLL) {
            unsigned long long so[GATHER_UNROLL], po[GATHER_UNROLL];
#pragma unroll
            for (int u = 0; u < GATHER_UNROLL; ++u) {
                const int from = min(r + u, 31);
                so[u] = __shfl_sync(0xFFFFFFFFu, src, from);
                po[u] = HOT ? __shfl_sync(0xFFFFFFFFu, pend, from) : NO_ROW;
                if (r + u >= rows) so[u] = NO_ROW;
            }
            for (uint32_t c = lane; c < L4; c += 32) {
                float4 a[GATHER_UNROLL], b[GATHER_UNROLL];
#pragma unroll
                for (int u = 0; u < GATHER_UNROLL; ++u) {
                    a[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (TWO) b[u] = a[u];
                    if (so[u] != NO_ROW) {
                        // with a hot tier, rows of non-replicated keys are unlikely to be read again soon:
                        // fetch them with the streaming hint so that they do not push the technique
                        // bitmap and the replicated rows out of L2
                        if (HOT && po[u] == NO_ROW) a[u] = ld_stream_v4(A.table + so[u] + c);
                        else a[u] = __ldg(A.table + so[u] + c);
                        if (TWO) b[u] = __ldg(B.table + so[u] + c);
                        if (HOT && po[u] != NO_ROW) {
                            a[u] = add_chunk<F64>(a[u], A.slab[po[u] + c]);
                            if (TWO) b[u] = add_chunk<F64>(b[u], B.slab[po[u] + c]);
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < GATHER_UNROLL; ++u) {
                    if (r + u < rows) {
                        const uint64_t oo = (base + r + u) * L4 + c;
                        st_stream_v4(A.out + oo, a[u]);
                        if (TWO) st_stream_v4(B.out + oo, b[u]);
                    }
                }
            }
        }
    }
}

// The same gather with 256-bit loads and stores, for one table whose rows are a multiple of 32 bytes and at most 32
// such chunks long, with 32 a multiple of the chunk count (64, 128 or 256 floats): a warp instruction then moves
// 32 / C8 whole rows, which halves the load/store instructions per byte.  Used when some keys are replicated: once
// many rows come from L2 (hot or repeated keys) the copy is bound by the instructions its rows take in the
// load/store pipe, not by DRAM.
template <bool HOT, int C8>
__global__ void __launch_bounds__(256, 4)
gather8_kernel(View v, const uint32_t* __restrict__ keys, uint64_t n, const float* __restrict__ table,
               const float* slab, float* __restrict__ out, int map, uint64_t map_base, uint64_t map_total, int do_count,
               uint32_t* __restrict__ keys_copy)
{
    grid_dependency_wait();
    constexpr int RPI = 32 / C8;                       // rows per warp instruction
    constexpr int UNR = 2;                             // instructions in flight
    const unsigned lane = threadIdx.x & 31;
    const unsigned sub = lane / C8, c = lane % C8;     // which of the instruction's rows, which chunk of it
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t nwarps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    const uint64_t L = (uint64_t)v.L4 * 4;
    const uint64_t stride = nwarps * 32;
    uint64_t base = warp * 32;
    const uint64_t end = n;
    uint32_t key_a = base + lane < end ? __ldg(keys + base + lane) : 0u;
    uint32_t key_b = base + stride + lane < end ? __ldg(keys + base + stride + lane) : 0u;
    uint32_t bits_a = (HOT && key_a < v.num_keys) ? __ldg(v.hot_bits + (key_a >> 5)) : 0u;
    for (; base < end; base += stride) {
        const uint64_t i = base + lane;
        const bool in = i < end;
        const uint32_t key = key_a;
        const uint32_t bits = bits_a;
        key_a = key_b;
        bits_a = (HOT && key_a < v.num_keys) ? __ldg(v.hot_bits + (key_a >> 5)) : 0u;
        key_b = base + 2 * stride + lane < end ? __ldg(keys + base + 2 * stride + lane) : 0u;
        const bool valid = in && key < v.num_keys;
        if (in && !valid) flag_bad_key(v);
        if (keys_copy && in) keys_copy[i] = key;                   // PullSample hands the keys out as well
        // row numbers instead of offsets: one 32-bit shuffle each; 0xFFFFFFFF = no such row
        uint32_t src = valid ? key : 0xFFFFFFFFu;
        uint32_t pend = 0xFFFFFFFFu;                    // replica row (worker * Hcap + slot) of a replicated key
        if (HOT && valid && ((bits >> (key & 31)) & 1u)) {
            const uint32_t slot = (uint32_t)__ldg(v.slot_of + key);
            const uint64_t idx = map_base + i;
            const uint32_t q = map == 0 ? worker_of_item(idx, map_total, v.R) : chunk_of_pos(idx, map_total, v.R);
            pend = q * (uint32_t)v.Hcap + slot;
        }
        if (do_count && v.count) {
            if (valid) atomicAdd(v.cnt + key, 1ull);
            unsigned hot_m = __ballot_sync(0xFFFFFFFFu, valid && pend != 0xFFFFFFFFu);
            unsigned cold_m = __ballot_sync(0xFFFFFFFFu, valid && pend == 0xFFFFFFFFu);
            if (lane == 0) {
                if (hot_m) atomicAdd(&v.st->hot_hits, (unsigned long long)__popc(hot_m));
                if (cold_m) atomicAdd(&v.st->cold_hits, (unsigned long long)__popc(cold_m));
            }
        }
        const int rows = (int)min((uint64_t)32, end - base);
        for (int r0 = 0; r0 < rows; r0 += UNR * RPI) {
            uint32_t so[UNR], po[UNR];
            F8 a[UNR];
#pragma unroll
            for (int u = 0; u < UNR; ++u) {
                const int row = r0 + u * RPI + (int)sub;
                so[u] = __shfl_sync(0xFFFFFFFFu, src, row & 31);
                po[u] = HOT ? __shfl_sync(0xFFFFFFFFu, pend, row & 31) : 0xFFFFFFFFu;
                if (row >= rows) so[u] = 0xFFFFFFFFu;
            }
#pragma unroll
            for (int u = 0; u < UNR; ++u) {
                a[u].a = make_float4(0.f, 0.f, 0.f, 0.f);
                a[u].b = a[u].a;
                if (so[u] != 0xFFFFFFFFu) {
                    const float* p = table + (uint64_t)so[u] * L + 8 * c;
                    // rows of non-replicated keys are unlikely to be read again soon: streaming hint
                    a[u] = (HOT && po[u] == 0xFFFFFFFFu) ? ld8_stream(p) : ld8_cached(p);
                    if (HOT && po[u] != 0xFFFFFFFFu) {
                        const F8 d = ld8_plain(slab + (uint64_t)po[u] * L + 8 * c);
                        a[u].a = add4(a[u].a, d.a);
                        a[u].b = add4(a[u].b, d.b);
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < UNR; ++u) {
                const int row = r0 + u * RPI + (int)sub;
                if (row < rows) st8_stream(out + (base + row) * L + 8 * c, a[u]);
            }
        }
    }
}

nups_status nups_gather_internal(nups_store* s, const uint32_t* d_keys, uint64_t n, float* d_out_val,
                                 float* d_out_acc, int worker_map, uint64_t map_base, uint64_t map_total,
                                 int do_count, cudaStream_t st, uint32_t* d_keys_copy)
{
    if (n == 0 || (!d_out_val && !d_out_acc)) return NUPS_OK;
    View v = nups_view(s);
    TablePair V = {(const float4*)s->val, (const float4*)s->dval, (float4*)d_out_val};
    TablePair C = {(const float4*)s->acc, (const float4*)s->dacc, (float4*)d_out_acc};
    const bool two = d_out_val && d_out_acc;
    TablePair A = d_out_val ? V : C, B = C;
    unsigned grid = grid_for(n, 32 * 8, (unsigned)s->sm_count * 4);     // 4 resident blocks per SM, grid-stride
    // one table, rows of 8, 16 or 32 chunks of 32 bytes, everything 32-byte aligned, some keys replicated: the
    // 256-bit variant.  (Measured on 1M-key pulls of 128-float rows: with a hot tier 152 vs 163 us at Zipf 1.0 and
    // 20-25 % faster when keys repeat as under sample reuse; without a hot tier, where every row comes from DRAM,
    // 187 vs 180 us, so those calls keep the 128-bit kernel.)
    const uint32_t c8 = s->L / 8;
    float* out1 = two ? nullptr : A.out ? (float*)A.out : nullptr;
    if (s->H && s->vb == 4 && !two && s->L % 8 == 0 && (c8 == 8 || c8 == 16 || c8 == 32) && ((uintptr_t)out1 & 31) == 0 &&
        (uint64_t)s->R * s->Hcap < 0xFFFFFFFFull) {
        const float* table = (const float*)A.table;
        const float* slab = (const float*)A.slab;
        nups_time_begin(s, st, worker_map == 1 ? NUPS_TIMED_SAMPLE_ROWS : NUPS_TIMED_PULL);
#define NUPS_G8(C8_)                                                                                                     \
        nups_launch_dependent(gather8_kernel<true, C8_>, grid, 256, 0, st, v, d_keys, n, table, slab, out1, worker_map, map_base, map_total, \
                                                        do_count, d_keys_copy)
        if (c8 == 8) NUPS_G8(8);
        else if (c8 == 16) NUPS_G8(16);
        else NUPS_G8(32);
#undef NUPS_G8
        nups_time_end(s, st);
        LAUNCH_CHECK(s);
        return NUPS_OK;
    }
    nups_time_begin(s, st, worker_map == 1 ? NUPS_TIMED_SAMPLE_ROWS : NUPS_TIMED_PULL);
#define NUPS_GATHER(HOT_, TWO_, F64_)                                                                                  \
    nups_launch_dependent(gather_kernel<HOT_, TWO_, F64_>, grid, 256, 0, st, v, d_keys, n, A, B, worker_map, map_base, map_total, do_count, \
                                                          d_keys_copy)
    if (s->vb == 8) {                        // only replica reads add; rows without a replica are copied whatever they hold
        if (s->H) { if (two) NUPS_GATHER(true, true, true); else NUPS_GATHER(true, false, true); }
        else { if (two) NUPS_GATHER(false, true, false); else NUPS_GATHER(false, false, false); }
    } else if (s->H) {
        if (two) NUPS_GATHER(true, true, false); else NUPS_GATHER(true, false, false);
    } else {
        if (two) NUPS_GATHER(false, true, false); else NUPS_GATHER(false, false, false);
    }
#undef NUPS_GATHER
    nups_time_end(s, st);
    LAUNCH_CHECK(s);
    return NUPS_OK;
}

extern "C" nups_status nups_pull2(nups_store* s, const uint32_t* d_keys, uint64_t n, void* d_out_val_, void* d_out_acc_,
                                  void* stream)
{
    float* d_out_val = (float*)d_out_val_;
    float* d_out_acc = (float*)d_out_acc_;
    if (!s || (n && !d_keys) || n >= (1ull << 32)) return NUPS_EINVAL;
    if (d_out_acc && !s->acc) return NUPS_EINVAL;
    if (n && !d_out_val && !d_out_acc) return NUPS_EINVAL;
    return nups_gather_internal(s, d_keys, n, d_out_val, d_out_acc, 0, 0, n, 1, (cudaStream_t)stream, nullptr);
}

extern "C" nups_status nups_pull(nups_store* s, const uint32_t* d_keys, uint64_t n, void* d_out, void* stream)
{
    if (n && !d_out) return NUPS_EINVAL;
    return nups_pull2(s, d_keys, n, d_out, nullptr, stream);
}

// ---------------------------------------------------------------------------------------------
// push, fast mode: 128-bit reductions straight to the destination row.  Within a window of 32
// rows, rows with the same destination are summed in registers first (__match_any_sync) so that
// a hot destination receives one reduction per window instead of one per row.
// TWO = a second table gets its own deltas from the same call.
// ---------------------------------------------------------------------------------------------
// Two rows in flight per warp and four resident blocks of 256 threads per multiprocessor (64 registers a thread): measured
// against four rows and three blocks (80 registers), the extra warps are worth more than the deeper unrolling at every skew
// (1M keys x 128 floats: 275 vs 279 us at s = 0, 195 vs 199 us at s = 1.0 with 1,000 replicated keys, 138 vs 152 us at s = 1.4).
constexpr int PUSH_UNROLL = 2;
constexpr int PUSH_THREADS = 256;
constexpr int PUSH_BLOCKS = 4;            // one table; calls that update two tables at once keep three (80 registers)

struct PushPair {
    const float4* delta;   // [n][L] updates
    float* table;          // stored rows
    float* slab;           // replica slabs
};

// TIER = the block keeps shared-memory accumulators for the hottest replica slots (slot < tier_rows)
// of ONE worker (block b serves worker b mod R and visits only that worker's share of the windows);
// updates to those slots are added in shared memory and reach the worker's replica once, when the
// block ends.  This is what keeps thousands of additions to one hot row from queueing at one L2
// address.
// TIER = 2: nothing is replicated, so there are no slots to key the accumulators on; the block then uses them as a
// direct-mapped cache of rows: accumulator (key mod tier_rows) is claimed by the first key that asks for it and
// takes that key's updates until the block ends (other keys that map there go straight to their rows).  Frequent
// keys show up early and often, so they take most accumulators, and a skewed batch stops queueing at a few L2
// addresses even when its frequent keys were never marked for replication.
template <bool HOT, bool TWO, int TIER, bool F64>
__global__ void __launch_bounds__(PUSH_THREADS, TWO ? PUSH_BLOCKS - 1 : PUSH_BLOCKS)
push_atomic_kernel(View v, const uint32_t* __restrict__ keys, uint64_t n, PushPair A, PushPair B, uint64_t n_items,
                   uint32_t rows_per_item, uint32_t tier_rows)
{
    grid_dependency_wait();
    extern __shared__ __align__(16) float tier_mem[];                  // TIER: [tier_rows][L] sums, then touched bits
    const unsigned lane = threadIdx.x & 31;
    const uint32_t L4 = v.L4;
    const uint32_t R = v.R;
    unsigned* touched = reinterpret_cast<unsigned*>(tier_mem + (size_t)tier_rows * L4 * 4);
    unsigned* tags = touched + (tier_rows + 31) / 32;                  // TIER == 2: key that owns each accumulator
    if (TIER) {
        float4* z = reinterpret_cast<float4*>(tier_mem);
        for (uint32_t e = threadIdx.x; e < tier_rows * L4; e += blockDim.x) z[e] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (uint32_t e = threadIdx.x; e < (tier_rows + 31) / 32; e += blockDim.x) touched[e] = 0u;
        if (TIER == 2)
            for (uint32_t e = threadIdx.x; e < tier_rows; e += blockDim.x) tags[e] = NUPS_INVALID_KEY;
        __syncthreads();
    }
    // Windows are visited in an order that interleaves the workers' chunks: the window range is cut
    // into R stretches of `per` windows; without the tier, slot u of the schedule is window
    // (u mod R) * per + u / R, so warps that run at the same time add to different replicas of a
    // hot key; with the tier, a block walks the stretch of its own worker only.
    const uint64_t W = (n + 31) / 32;
    const uint64_t per = (W + R - 1) / R;
    const uint32_t my_q = TIER == 1 ? blockIdx.x % R : 0u;
    const uint64_t warp = TIER == 1 ? ((uint64_t)(blockIdx.x / R) * blockDim.x + threadIdx.x) >> 5
                               : ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t nwarps = TIER == 1 ? ((uint64_t)(gridDim.x / R) * blockDim.x) >> 5 : ((uint64_t)gridDim.x * blockDim.x) >> 5;
    const uint64_t slots = TIER == 1 ? per : per * R;
    auto window_of = [&](uint64_t u) -> uint64_t {
        if (u >= slots) return W;
        const uint64_t w = TIER == 1 ? (uint64_t)my_q * per + u : (u % R) * per + u / R;
        return (w < W) ? w : W;
    };
    auto load_key = [&](uint64_t w) -> uint32_t {
        return (w < W && w * 32 + lane < n) ? __ldg(keys + w * 32 + lane) : NUPS_INVALID_KEY;
    };
    // lookups run two windows ahead of the reductions
    uint64_t win_a = window_of(warp), win_b = window_of(warp + nwarps);
    uint32_t key_a = load_key(win_a), key_b = load_key(win_b);
    uint32_t bits_a = (HOT && key_a < v.num_keys) ? __ldg(v.hot_bits + (key_a >> 5)) : 0u;
    for (uint64_t u = warp; u < slots; u += nwarps) {
        const uint64_t win = win_a;
        const uint32_t key = key_a;
        const uint32_t bits = bits_a;
        win_a = win_b; key_a = key_b;
        bits_a = (HOT && key_a < v.num_keys) ? __ldg(v.hot_bits + (key_a >> 5)) : 0u;
        win_b = window_of(u + 2 * nwarps);
        key_b = load_key(win_b);
        if (win >= W) continue;
        const uint64_t base = win * 32;
        const uint64_t i = base + lane;
        const bool in = i < n;
        const bool valid = in && key < v.num_keys;
        if (in && !valid) flag_bad_key(v);
        // destination: row offset in floats, lowest bit set when it lies in the replica slab
        unsigned long long dest = NO_ROW - lane;          // invalid rows: a value no other lane has
        bool hot = false;
        size_t hrow = 0;
        int tier = -1;                                    // shared-memory accumulator of this row, if any
        if (valid) {
            dest = ((unsigned long long)key * L4) << 3;
            if (HOT && ((bits >> (key & 31)) & 1u)) {
                hot = true;
                const uint32_t slot = (uint32_t)__ldg(v.slot_of + key);
                const uint32_t q = rows_per_item == 1 ? worker_of_item(i, n_items, R)
                                                      : worker_of_item(i / rows_per_item, n_items, R);
                dest = ((((unsigned long long)q * v.Hcap + slot) * L4) << 3) | 1ull;
                hrow = (size_t)q * v.Hcap + slot;
                if (TIER == 1 && slot < tier_rows && q == my_q) tier = (int)slot;
            }
            if (TIER == 2) {
                const uint32_t at = key % tier_rows;
                uint32_t owner = tags[at];
                if (owner == NUPS_INVALID_KEY) {
                    owner = atomicCAS(&tags[at], NUPS_INVALID_KEY, key);
                    if (owner == NUPS_INVALID_KEY) owner = key;
                }
                if (owner == key) tier = (int)at;
            }
        }
        if (v.count) {
            if (valid) atomicAdd(v.cnt + key, 1ull);
            unsigned hot_m = __ballot_sync(0xFFFFFFFFu, valid && hot);
            unsigned cold_m = __ballot_sync(0xFFFFFFFFu, valid && !hot);
            if (lane == 0) {
                if (hot_m) atomicAdd(&v.st->hot_hits, (unsigned long long)__popc(hot_m));
                if (cold_m) atomicAdd(&v.st->cold_hits, (unsigned long long)__popc(cold_m));
            }
        }
        const unsigned grp = __match_any_sync(0xFFFFFFFFu, dest);
        const bool leader = valid && (lane == (unsigned)(__ffs(grp) - 1));
        // mark the slot as touched: one lane per destination, and only if nobody has yet (a hot slot would
        // otherwise take hundreds of thousands of stores to one address)
        if (HOT && leader && hot) {
            uint32_t* flag = v.dirty + hrow;          // replica row index = q * Hcap + slot
            if (*flag == 0u) *flag = 1u;
        }
        unsigned singles = __ballot_sync(0xFFFFFFFFu, leader && __popc(grp) == 1);
        unsigned multis = __ballot_sync(0xFFFFFFFFu, leader && __popc(grp) > 1);

        // rows that are alone in their window: PUSH_UNROLL at a time
        while (singles) {
            int src[PUSH_UNROLL], tr[PUSH_UNROLL];
            unsigned long long de[PUSH_UNROLL];
#pragma unroll
            for (int u4 = 0; u4 < PUSH_UNROLL; ++u4) {
                src[u4] = singles ? __ffs(singles) - 1 : -1;
                singles &= singles - 1;
                de[u4] = __shfl_sync(0xFFFFFFFFu, dest, src[u4] < 0 ? 0 : src[u4]);
                tr[u4] = TIER ? __shfl_sync(0xFFFFFFFFu, tier, src[u4] < 0 ? 0 : src[u4]) : -1;
            }
            for (uint32_t c = lane; c < L4; c += 32) {
                float4 a[PUSH_UNROLL], b[PUSH_UNROLL];
#pragma unroll
                for (int u4 = 0; u4 < PUSH_UNROLL; ++u4) {
                    if (src[u4] >= 0) {
                        const uint64_t in_off = (base + src[u4]) * L4 + c;
                        a[u4] = ld_stream_v4(A.delta + in_off);
                        if (TWO) b[u4] = ld_stream_v4(B.delta + in_off);
                    }
                }
#pragma unroll
                for (int u4 = 0; u4 < PUSH_UNROLL; ++u4) {
                    if (src[u4] >= 0) {
                        if (TIER && tr[u4] >= 0) {
                            // accumulator rows are stored component by component, [4][L4], so that the 32
                            // lanes of one addition fall into 32 different banks
                            float* t = tier_mem + (size_t)tr[u4] * L4 * 4 + c;
                            atomicAdd(t, a[u4].x); atomicAdd(t + L4, a[u4].y); atomicAdd(t + 2 * L4, a[u4].z);
                            atomicAdd(t + 3 * L4, a[u4].w);
                        } else {
                            const bool h = HOT && (de[u4] & 1ull);
                            const uint64_t off = (de[u4] >> 3) * 4 + (uint64_t)c * 4;
                            red_add_chunk<F64>((h ? A.slab : A.table) + off, a[u4]);
                            if (TWO) red_add_chunk<F64>((h ? B.slab : B.table) + off, b[u4]);
                        }
                    }
                }
            }
            if (TIER && lane == 0) {
#pragma unroll
                for (int u4 = 0; u4 < PUSH_UNROLL; ++u4)
                    if (src[u4] >= 0 && tr[u4] >= 0 && !((touched[tr[u4] >> 5] >> (tr[u4] & 31)) & 1u))
                        atomicOr(&touched[tr[u4] >> 5], 1u << (tr[u4] & 31));
            }
        }
        // destinations hit more than once in the window: sum the members (loads PUSH_UNROLL at a time), one reduction
        while (multis) {
            const int ld = __ffs(multis) - 1;
            multis &= multis - 1;
            const unsigned members = __shfl_sync(0xFFFFFFFFu, grp, ld);
            const unsigned long long de = __shfl_sync(0xFFFFFFFFu, dest, ld);
            const int tr = TIER ? __shfl_sync(0xFFFFFFFFu, tier, ld) : -1;
            const bool h = HOT && (de & 1ull);
            for (uint32_t c = lane; c < L4; c += 32) {
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
                unsigned mm = members;
                while (mm) {
                    int m[PUSH_UNROLL];
                    float4 x[PUSH_UNROLL], y[PUSH_UNROLL];
#pragma unroll
                    for (int u4 = 0; u4 < PUSH_UNROLL; ++u4) {
                        m[u4] = mm ? __ffs(mm) - 1 : -1;
                        mm &= mm - 1;
                    }
#pragma unroll
                    for (int u4 = 0; u4 < PUSH_UNROLL; ++u4) {
                        if (m[u4] >= 0) {
                            const uint64_t in_off = (base + m[u4]) * L4 + c;
                            x[u4] = ld_stream_v4(A.delta + in_off);
                            if (TWO) y[u4] = ld_stream_v4(B.delta + in_off);
                        }
                    }
#pragma unroll
                    for (int u4 = 0; u4 < PUSH_UNROLL; ++u4) {
                        if (m[u4] >= 0) {
                            a = add_chunk<F64>(a, x[u4]);
                            if (TWO) b = add_chunk<F64>(b, y[u4]);
                        }
                    }
                }
                if (TIER && tr >= 0) {
                    float* t = tier_mem + (size_t)tr * L4 * 4 + c;
                    atomicAdd(t, a.x); atomicAdd(t + L4, a.y); atomicAdd(t + 2 * L4, a.z); atomicAdd(t + 3 * L4, a.w);
                } else {
                    const uint64_t off = (de >> 3) * 4 + (uint64_t)c * 4;
                    red_add_chunk<F64>((h ? A.slab : A.table) + off, a);
                    if (TWO) red_add_chunk<F64>((h ? B.slab : B.table) + off, b);
                }
            }
            if (TIER && tr >= 0 && lane == 0 && !((touched[tr >> 5] >> (tr & 31)) & 1u))
                atomicOr(&touched[tr >> 5], 1u << (tr & 31));
        }
    }
    if (TIER) {
        // hand the block's sums to the worker's replica: one reduction per touched row
        __syncthreads();
        for (uint32_t sl = threadIdx.x >> 5; sl < tier_rows; sl += blockDim.x >> 5) {
            if (!((touched[sl >> 5] >> (sl & 31)) & 1u)) continue;
            float* dst = TIER == 2 ? A.table + (size_t)tags[sl] * L4 * 4 : A.slab + ((size_t)my_q * v.Hcap + sl) * L4 * 4;
            const float* t = tier_mem + (size_t)sl * L4 * 4;
            for (uint32_t c = lane; c < L4; c += 32)
                red_add_v4(dst + (size_t)c * 4, make_float4(t[c], t[c + L4], t[c + 2 * L4], t[c + 3 * L4]));
        }
    }
}

// ---------------------------------------------------------------------------------------------
// push, deterministic mode: rows are sorted (stably) by destination, then one warp per
// destination adds its rows one by one in input order.
// ---------------------------------------------------------------------------------------------
template <bool HOT>
__global__ void push_dest_kernel(View v, const uint32_t* __restrict__ keys, uint64_t n, uint64_t n_items,
                                 uint32_t rows_per_item, unsigned long long invalid_dest,
                                 unsigned long long* __restrict__ dest, uint32_t* __restrict__ idx)
{
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned lane = threadIdx.x & 31;
    bool in = i < n;
    uint32_t key = in ? keys[i] : 0u;
    bool valid = in && key < v.num_keys;
    if (in && !valid) flag_bad_key(v);
    bool hot = false;
    unsigned long long d = invalid_dest;
    if (valid) {
        d = key;
        if (HOT && key_is_hot(v, key)) {
            hot = true;
            uint32_t slot = (uint32_t)v.slot_of[key];
            uint32_t q = worker_of_item(i / rows_per_item, n_items, v.R);
            d = (1ull << 32) + (unsigned long long)q * v.H + slot;
            if (v.dirty[(size_t)q * v.Hcap + slot] == 0u) v.dirty[(size_t)q * v.Hcap + slot] = 1u;
        }
    }
    if (in) { dest[i] = d; idx[i] = (uint32_t)i; }
    if (v.count) {
        if (valid) atomicAdd(v.cnt + key, 1ull);
        unsigned hot_m = __ballot_sync(0xFFFFFFFFu, valid && hot);
        unsigned cold_m = __ballot_sync(0xFFFFFFFFu, valid && !hot);
        if (lane == 0) {
            if (hot_m) atomicAdd(&v.st->hot_hits, (unsigned long long)__popc(hot_m));
            if (cold_m) atomicAdd(&v.st->cold_hits, (unsigned long long)__popc(cold_m));
        }
    }
}

template <bool F64>
__global__ void __launch_bounds__(256)
push_ordered_kernel(View v, const unsigned long long* __restrict__ dest, const uint32_t* __restrict__ idx, uint64_t n,
                    unsigned long long invalid_dest, const float4* __restrict__ dv, const float4* __restrict__ da)
{
    const unsigned lane = threadIdx.x & 31;
    const uint64_t j = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (j >= n) return;
    unsigned long long d = dest[j];
    if (d == invalid_dest) return;
    if (j > 0 && dest[j - 1] == d) return;           // not the first row of its destination
    const uint32_t L4 = v.L4;
    float4* tv;
    float4* ta;
    if (d >> 32) {
        unsigned long long r = d - (1ull << 32);
        uint64_t q = r / v.H, slot = r % v.H;
        uint64_t off = (q * v.Hcap + slot) * L4;
        tv = (float4*)v.dval + off;
        ta = (float4*)v.dacc + off;
    } else {
        tv = (float4*)v.val + d * L4;
        ta = (float4*)v.acc + d * L4;
    }
    uint64_t end = j + 1;
    while (end < n && dest[end] == d) ++end;
    for (uint32_t c = lane; c < L4; c += 32) {
        float4 a = dv ? tv[c] : make_float4(0.f, 0.f, 0.f, 0.f);
        float4 b = da ? ta[c] : make_float4(0.f, 0.f, 0.f, 0.f);
        uint64_t p = j;
        for (; p + 4 <= end; p += 4) {               // loads issued together, adds kept in order
            uint64_t o0 = (uint64_t)idx[p] * L4 + c, o1 = (uint64_t)idx[p + 1] * L4 + c;
            uint64_t o2 = (uint64_t)idx[p + 2] * L4 + c, o3 = (uint64_t)idx[p + 3] * L4 + c;
            if (dv) {
                float4 x0 = dv[o0], x1 = dv[o1], x2 = dv[o2], x3 = dv[o3];
                a = add_chunk<F64>(add_chunk<F64>(add_chunk<F64>(add_chunk<F64>(a, x0), x1), x2), x3);
            }
            if (da) {
                float4 y0 = da[o0], y1 = da[o1], y2 = da[o2], y3 = da[o3];
                b = add_chunk<F64>(add_chunk<F64>(add_chunk<F64>(add_chunk<F64>(b, y0), y1), y2), y3);
            }
        }
        for (; p < end; ++p) {
            uint64_t o = (uint64_t)idx[p] * L4 + c;
            if (dv) a = add_chunk<F64>(a, dv[o]);
            if (da) b = add_chunk<F64>(b, da[o]);
        }
        if (dv) tv[c] = a;
        if (da) ta[c] = b;
    }
}

static int bits_for(unsigned long long maxval)
{
    int b = 1;
    while (b < 64 && (maxval >> b)) ++b;
    return b;
}

size_t nups_push_scratch_bytes(const nups_store* s, uint64_t n)
{
    if (!s->cfg.deterministic) return 0;
    return 2 * align256(n * 8) + 2 * align256(n * 4) + nups_sort_scratch_bytes(n);
}

nups_status nups_push_internal(nups_store* s, const uint32_t* d_keys, uint64_t n, uint32_t rows_per_item,
                               const float* d_dval, const float* d_dacc, cudaStream_t st)
{
    char* sc = nullptr;
    if (s->cfg.deterministic && n) {
        nups_status rc = nups_scratch(s, nups_push_scratch_bytes(s, n), &sc);
        if (rc != NUPS_OK) return rc;
    }
    return nups_push_with_scratch(s, d_keys, n, rows_per_item, d_dval, d_dacc, sc, st);
}

nups_status nups_push_with_scratch(nups_store* s, const uint32_t* d_keys, uint64_t n, uint32_t rows_per_item,
                                   const float* d_dval, const float* d_dacc, char* sc, cudaStream_t st)
{
    if (n == 0 || (!d_dval && !d_dacc)) return NUPS_OK;
    View v = nups_view(s);
    uint64_t n_items = n / rows_per_item;
    if (!s->cfg.deterministic) {
        const bool two = d_dval && d_dacc;
        unsigned grid = grid_for(n, PUSH_THREADS, (unsigned)s->sm_count * (two ? PUSH_BLOCKS - 1 : PUSH_BLOCKS));  // resident at once, grid-stride
        PushPair V = {(const float4*)d_dval, s->val, s->dval};
        PushPair C = {(const float4*)d_dacc, s->acc, s->dacc};
        PushPair A = d_dval ? V : C, B = C;
        // shared-memory tier: single-table calls with replicated keys, enough blocks to give every worker some
        uint32_t tier_rows = 0;
        size_t tier_bytes = 0;
        const bool cache = !s->H && !two && n >= 32768 && s->vb == 4;  // no replicated keys: accumulators as a row cache
        if ((s->H && !two && rows_per_item == 1 && grid >= s->R && n >= 32768 && s->vb == 4) || cache) {
            const size_t row_bytes = (size_t)s->L * 4;
            size_t budget = (size_t)(192 / PUSH_BLOCKS) * 1024;                 // the blocks of a multiprocessor share 192 KB
            const size_t per_row = row_bytes + (cache ? 4 : 0) + 1;    // sums, owner tag, touched bit (rounded up)
            tier_rows = s->cfg.smem_hot_rows ? s->cfg.smem_hot_rows : (uint32_t)(budget / per_row);
            if (tier_rows > budget / per_row) tier_rows = (uint32_t)(budget / per_row);
            if (cache && tier_rows > 1024) tier_rows = 1024;
            if (!cache && tier_rows > s->H) tier_rows = (uint32_t)s->H;
            tier_bytes = tier_rows * row_bytes + ((tier_rows + 31) / 32) * 4 + (cache ? tier_rows * 4 : 0);
            if (tier_rows && !s->push_smem_opted) {
                CK(cudaFuncSetAttribute(push_atomic_kernel<true, false, 1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)(budget + 2048)));
                CK(cudaFuncSetAttribute(push_atomic_kernel<false, false, 2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)(budget + 2048)));
                s->push_smem_opted = true;
            }
        }
        nups_time_begin(s, st, NUPS_TIMED_PUSH);
        if (tier_rows && cache) {
            nups_launch_dependent(push_atomic_kernel<false, false, 2, false>, grid, PUSH_THREADS, tier_bytes, st, v, d_keys, n, A, B, n_items, rows_per_item,
                                                                             tier_rows);
        } else if (tier_rows) {
            grid = grid / s->R * s->R;              // every worker gets the same number of blocks
            nups_launch_dependent(push_atomic_kernel<true, false, 1, false>, grid, PUSH_THREADS, tier_bytes, st, v, d_keys, n, A, B, n_items, rows_per_item,
                                                                             tier_rows);
        } else {
#define NUPS_PUSH0(HOT_, TWO_, F64_) \
    nups_launch_dependent(push_atomic_kernel<HOT_, TWO_, 0, F64_>, grid, PUSH_THREADS, 0, st, v, d_keys, n, A, B, n_items, rows_per_item, 0)
            if (s->vb == 8) {
                if (s->H) { if (two) NUPS_PUSH0(true, true, true); else NUPS_PUSH0(true, false, true); }
                else { if (two) NUPS_PUSH0(false, true, true); else NUPS_PUSH0(false, false, true); }
            } else if (s->H) {
                if (two) NUPS_PUSH0(true, true, false); else NUPS_PUSH0(true, false, false);
            } else {
                if (two) NUPS_PUSH0(false, true, false); else NUPS_PUSH0(false, false, false);
            }
#undef NUPS_PUSH0
        }
        nups_time_end(s, st);
        LAUNCH_CHECK(s);
        return NUPS_OK;
    }
    unsigned long long invalid_dest = s->H ? (1ull << 32) + (unsigned long long)s->R * s->H : s->num_keys;
    int bits = bits_for(invalid_dest);
    nups_status rc;
    unsigned long long* k0 = (unsigned long long*)sc; sc += align256(n * 8);
    unsigned long long* k1 = (unsigned long long*)sc; sc += align256(n * 8);
    uint32_t* v0 = (uint32_t*)sc; sc += align256(n * 4);
    uint32_t* v1 = (uint32_t*)sc; sc += align256(n * 4);
    if (s->H)
        push_dest_kernel<true><<<grid_for(n, 256), 256, 0, st>>>(v, d_keys, n, n_items, rows_per_item, invalid_dest, k0, v0);
    else
        push_dest_kernel<false><<<grid_for(n, 256), 256, 0, st>>>(v, d_keys, n, n_items, rows_per_item, invalid_dest, k0, v0);
    LAUNCH_CHECK(s);
    rc = nups_sort_pairs(s, k0, v0, k1, v1, n, bits, sc, st);
    if (rc != NUPS_OK) return rc;
    if (s->vb == 8)
        push_ordered_kernel<true><<<grid_for(n * 32, 256), 256, 0, st>>>(v, k1, v1, n, invalid_dest, (const float4*)d_dval,
                                                                         (const float4*)d_dacc);
    else
        push_ordered_kernel<false><<<grid_for(n * 32, 256), 256, 0, st>>>(v, k1, v1, n, invalid_dest, (const float4*)d_dval,
                                                                          (const float4*)d_dacc);
    LAUNCH_CHECK(s);
    return NUPS_OK;
}

extern "C" nups_status nups_push2(nups_store* s, const uint32_t* d_keys, uint64_t n, const void* d_dval_,
                                  const void* d_dacc_, void* stream)
{
    const float* d_dval = (const float*)d_dval_;
    const float* d_dacc = (const float*)d_dacc_;
    if (!s || (n && !d_keys) || n >= (1ull << 32)) return NUPS_EINVAL;
    if (d_dacc && !s->acc) return NUPS_EINVAL;
    if (n && !d_dval && !d_dacc) return NUPS_EINVAL;
    return nups_push_internal(s, d_keys, n, 1, d_dval, d_dacc, (cudaStream_t)stream);
}

extern "C" nups_status nups_push(nups_store* s, const uint32_t* d_keys, uint64_t n, const void* d_delta, void* stream)
{
    if (n && !d_delta) return NUPS_EINVAL;
    return nups_push2(s, d_keys, n, d_delta, nullptr, stream);
}

// ---------------------------------------------------------------------------------------------
// sync: merge the workers' pending updates of every touched hot slot into the stored row,
// worker 0 first, and clear them.
// ---------------------------------------------------------------------------------------------
template <bool F64>
__global__ void sync_kernel(View v, const uint32_t* __restrict__ hot_keys)
{
    grid_dependency_wait();
    const uint32_t L4 = v.L4;
    uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint64_t total = (uint64_t)v.H * L4;
    if (t >= total) return;
    uint32_t slot = (uint32_t)(t / L4), c = (uint32_t)(t % L4);
    // only replicas that were written since the last sync are read, added (worker 0 first) and cleared
    bool any = false;
    for (uint32_t r = 0; r < v.R; ++r) any = any || v.dirty[(size_t)r * v.Hcap + slot] != 0u;
    if (!any) return;
    uint32_t key = hot_keys[slot];
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int which = 0; which < 2; ++which) {
        float4* table = (float4*)(which ? v.acc : v.val);
        float4* slab = (float4*)(which ? v.dacc : v.dval);
        if (!table || !slab) continue;
        float4 sum = zero;
        for (uint32_t r0 = 0; r0 < v.R; r0 += 4) {
            float4 x[4];
            bool d[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                d[u] = r0 + u < v.R && v.dirty[(size_t)(r0 + u) * v.Hcap + slot] != 0u;
                if (d[u]) x[u] = slab[((uint64_t)(r0 + u) * v.Hcap + slot) * L4 + c];
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (d[u]) {
                    sum = add_chunk<F64>(sum, x[u]);
                    slab[((uint64_t)(r0 + u) * v.Hcap + slot) * L4 + c] = zero;
                }
            }
        }
        if (v.merge_mean) {                                   // the mean over the workers that touched the slot
            uint32_t touched = 0;
            for (uint32_t r = 0; r < v.R; ++r) touched += v.dirty[(size_t)r * v.Hcap + slot] != 0u;
            if (F64) {
                const double2 d = as_d2(sum);
                sum = as_f4(make_double2(__ddiv_rn(d.x, (double)touched), __ddiv_rn(d.y, (double)touched)));
            } else {
                const float by = (float)touched;
                sum = make_float4(__fdiv_rn(sum.x, by), __fdiv_rn(sum.y, by), __fdiv_rn(sum.z, by), __fdiv_rn(sum.w, by));
            }
        }
        float4* row = table + (uint64_t)key * L4 + c;
        *row = add_chunk<F64>(*row, sum);
    }
}

nups_status nups_sync_internal(nups_store* s, cudaStream_t st)
{
    if (s->H == 0) return NUPS_OK;        // nothing replicated: no work at all
    View v = nups_view(s);
    nups_background_begin(s, st);
    if (s->vb == 8) nups_launch_dependent(sync_kernel<true>, grid_for(s->H * (s->L / 4), 256), 256, 0, st, v, s->hot_keys);
    else nups_launch_dependent(sync_kernel<false>, grid_for(s->H * (s->L / 4), 256), 256, 0, st, v, s->hot_keys);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaMemsetAsync(s->dirty, 0, (size_t)s->R * s->Hcap * sizeof(uint32_t), st);
    nups_background_end(s, st);
    if (e != cudaSuccess) return nups_cuda_fail(e, "replica merge");
    s->launches++;
    s->syncs++;
    return NUPS_OK;
}

extern "C" nups_status nups_sync(nups_store* s, void* stream)
{
    if (!s) return NUPS_EINVAL;
    return nups_sync_internal(s, (cudaStream_t)stream);
}

// ---------------------------------------------------------------------------------------------
// access counting and hot-set selection
// ---------------------------------------------------------------------------------------------
__global__ void count_kernel(View v, const uint32_t* __restrict__ keys, uint64_t n)
{
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned lane = threadIdx.x & 31;
    bool in = i < n;
    uint32_t key = in ? keys[i] : 0u;
    bool valid = in && key < v.num_keys;
    if (in && !valid) flag_bad_key(v);
    unsigned long long tag = valid ? (unsigned long long)key : (~0ull - lane);
    unsigned grp = __match_any_sync(0xFFFFFFFFu, tag);
    if (valid && lane == (unsigned)(__ffs(grp) - 1)) atomicAdd(v.cnt + key, (unsigned long long)__popc(grp));
}

extern "C" nups_status nups_count_accesses(nups_store* s, const uint32_t* d_keys, uint64_t n, void* stream)
{
    if (!s || (n && !d_keys)) return NUPS_EINVAL;
    if (n == 0) return NUPS_OK;
    count_kernel<<<grid_for(n, 256), 256, 0, (cudaStream_t)stream>>>(nups_view(s), d_keys, n);
    LAUNCH_CHECK(s);
    return NUPS_OK;
}

extern "C" nups_status nups_get_counts(nups_store* s, uint64_t* d_out, void* stream)
{
    if (!s || !d_out) return NUPS_EINVAL;
    CK(cudaMemcpyAsync(d_out, s->cnt, s->num_keys * 8, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return NUPS_OK;
}

__global__ void count_sum_max_kernel(const unsigned long long* __restrict__ cnt, uint64_t n, DevStat* st)
{
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    unsigned long long sum = 0, mx = 0;
    for (; i < n; i += stride) {
        unsigned long long c = cnt[i];
        sum += c;
        mx = c > mx ? c : mx;
    }
    for (int o = 16; o > 0; o >>= 1) {
        sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
        unsigned long long m2 = __shfl_xor_sync(0xFFFFFFFFu, mx, o);
        mx = m2 > mx ? m2 : mx;
    }
    if ((threadIdx.x & 31) == 0) {
        atomicAdd(&st->tmp[0], sum);
        atomicMax(&st->tmp[1], mx);
    }
}

// flag[k] = 1 when key k is selected by the threshold rule cnt*num_keys > factor*total (exact)
__global__ void threshold_flag_kernel(const unsigned long long* __restrict__ cnt, uint64_t n, unsigned long long factor,
                                      unsigned long long total, unsigned long long* __restrict__ flag)
{
    uint64_t k = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= n) return;
    unsigned long long c = cnt[k];
    unsigned long long lhi = __umul64hi(c, n), llo = c * n;
    unsigned long long rhi = __umul64hi(factor, total), rlo = factor * total;
    flag[k] = (lhi > rhi || (lhi == rhi && llo > rlo)) ? 1ull : 0ull;
}

// composite sort key: (max_cnt - cnt) in the high part, key in the low `key_bits` bits, so that an
// ascending sort gives count descending, key ascending
__global__ void composite_kernel(const unsigned long long* __restrict__ cnt, uint64_t n, unsigned long long max_cnt,
                                 int key_bits, const unsigned long long* __restrict__ flag /* nullable */,
                                 const unsigned long long* __restrict__ pos /* exclusive scan of flag */,
                                 unsigned long long* __restrict__ comp, uint32_t* __restrict__ payload)
{
    uint64_t k = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= n) return;
    uint64_t o = k;
    if (flag) {
        if (!flag[k]) return;
        o = pos[k];
    }
    comp[o] = ((max_cnt - cnt[k]) << key_bits) | k;
    payload[o] = (uint32_t)k;
}

extern "C" nups_status nups_select_hot(nups_store* s, int by_topk, uint64_t param, uint32_t* d_keys_out,
                                       uint64_t* h_n_out, void* stream)
{
    if (!s || !d_keys_out || !h_n_out) return NUPS_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    uint64_t n = s->num_keys;
    *h_n_out = 0;
    CK(cudaMemsetAsync(&s->st->tmp[0], 0, 16, st));
    count_sum_max_kernel<<<grid_for(n, 256, (unsigned)s->sm_count * 8), 256, 0, st>>>(s->cnt, n, s->st);
    LAUNCH_CHECK(s);
    unsigned long long sm[2];
    CK(cudaMemcpyAsync(sm, &s->st->tmp[0], 16, cudaMemcpyDeviceToHost, st));
    CK(cudaStreamSynchronize(st));
    unsigned long long total = sm[0], max_cnt = sm[1];
    int key_bits = bits_for(n - 1), cnt_bits = bits_for(max_cnt);
    if (key_bits + cnt_bits > 64) return NUPS_ESTATE;
    size_t need = 4 * align256(n * 8) + 2 * align256(n * 4) + nups_sort_scratch_bytes(n) + nups_scan_scratch_bytes(n) + 256;
    char* sc;
    nups_status rc = nups_scratch(s, need, &sc);
    if (rc != NUPS_OK) return rc;
    unsigned long long* flag = (unsigned long long*)sc; sc += align256(n * 8);
    unsigned long long* pos = (unsigned long long*)sc; sc += align256(n * 8);
    unsigned long long* c0 = (unsigned long long*)sc; sc += align256(n * 8);
    unsigned long long* c1 = (unsigned long long*)sc; sc += align256(n * 8);
    uint32_t* p0 = (uint32_t*)sc; sc += align256(n * 4);
    uint32_t* p1 = (uint32_t*)sc; sc += align256(n * 4);
    unsigned long long* d_m = (unsigned long long*)sc; sc += 256;
    uint64_t m = n;
    if (!by_topk) {
        threshold_flag_kernel<<<grid_for(n, 256), 256, 0, st>>>(s->cnt, n, param, total, flag);
        LAUNCH_CHECK(s);
        rc = nups_scan_u64(s, flag, pos, n, d_m, sc, st);
        if (rc != NUPS_OK) return rc;
        unsigned long long hm = 0;
        CK(cudaMemcpyAsync(&hm, d_m, 8, cudaMemcpyDeviceToHost, st));
        CK(cudaStreamSynchronize(st));
        m = hm;
        if (m == 0) return NUPS_OK;
        composite_kernel<<<grid_for(n, 256), 256, 0, st>>>(s->cnt, n, max_cnt, key_bits, flag, pos, c0, p0);
    } else {
        if (param == 0) return NUPS_OK;
        composite_kernel<<<grid_for(n, 256), 256, 0, st>>>(s->cnt, n, max_cnt, key_bits, nullptr, nullptr, c0, p0);
    }
    LAUNCH_CHECK(s);
    char* sort_sc = sc + nups_scan_scratch_bytes(n);
    rc = nups_sort_pairs(s, c0, p0, c1, p1, m, key_bits + cnt_bits, sort_sc, st);
    if (rc != NUPS_OK) return rc;
    uint64_t take = by_topk ? (param < m ? param : m) : m;
    CK(cudaMemcpyAsync(d_keys_out, p1, take * 4, cudaMemcpyDeviceToDevice, st));
    CK(cudaStreamSynchronize(st));
    *h_n_out = take;
    return NUPS_OK;
}

// ---------------------------------------------------------------------------------------------
// per-key management
// ---------------------------------------------------------------------------------------------
// REPLICATE, pass 1: every listed key that is not hot yet is claimed by its first list position.
// slot_of holds: >= 0 hot slot; -1 single; <= -2 a claim by list position p encoded as -(p + 2).
__global__ void claim_kernel(int* slot_of, uint64_t num_keys, const uint32_t* __restrict__ keys, uint64_t n, DevStat* st)
{
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    uint32_t k = keys[i];
    if (k >= num_keys) { atomicCAS(&st->status, 0, NUPS_EKEY); return; }
    int mine = -(int)(i + 2);
    int cur = slot_of[k];
    while (cur < 0 && (cur == -1 || cur < mine)) {          // smaller position = larger (closer to -2) code
        int prev = atomicCAS(&slot_of[k], cur, mine);
        if (prev == cur) break;
        cur = prev;
    }
}
__global__ void winner_flag_kernel(const int* __restrict__ slot_of, uint64_t num_keys, const uint32_t* __restrict__ keys,
                                   uint64_t n, unsigned long long* __restrict__ flag)
{
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    uint32_t k = keys[i];
    flag[i] = (k < num_keys && slot_of[k] == -(int)(i + 2)) ? 1ull : 0ull;
}
__global__ void assign_slots_kernel(int* slot_of, uint32_t* hot_bits, uint32_t* hot_keys, const uint32_t* __restrict__ keys,
                                    uint64_t n, const unsigned long long* __restrict__ flag,
                                    const unsigned long long* __restrict__ pos, uint64_t H_old)
{
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n || !flag[i]) return;
    uint32_t k = keys[i];
    uint64_t slot = H_old + pos[i];
    slot_of[k] = (int)slot;
    hot_keys[slot] = k;
    atomicOr(&hot_bits[k >> 5], 1u << (k & 31));
}
// SINGLE: drop the listed keys, then renumber the surviving slots in their old order.
__global__ void demote_kernel(int* slot_of, uint32_t* hot_bits, uint64_t num_keys, const uint32_t* __restrict__ keys,
                              uint64_t n, DevStat* st)
{
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    uint32_t k = keys[i];
    if (k >= num_keys) { atomicCAS(&st->status, 0, NUPS_EKEY); return; }
    slot_of[k] = -1;
    atomicAnd(&hot_bits[k >> 5], ~(1u << (k & 31)));
}
__global__ void alive_flag_kernel(const int* __restrict__ slot_of, const uint32_t* __restrict__ hot_keys, uint64_t H,
                                  unsigned long long* __restrict__ flag)
{
    uint64_t sl = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (sl >= H) return;
    flag[sl] = slot_of[hot_keys[sl]] >= 0 ? 1ull : 0ull;
}
__global__ void renumber_kernel(int* slot_of, const uint32_t* __restrict__ hot_keys, uint32_t* __restrict__ hot_keys_new,
                                uint64_t H, const unsigned long long* __restrict__ flag,
                                const unsigned long long* __restrict__ pos)
{
    uint64_t sl = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (sl >= H || !flag[sl]) return;
    uint32_t k = hot_keys[sl];
    slot_of[k] = (int)pos[sl];
    hot_keys_new[pos[sl]] = k;
}

static nups_status grow_hot(nups_store* s, uint64_t need)
{
    if (need <= s->Hcap) return NUPS_OK;
    uint64_t cap = need + need / 4 + 16;
    uint32_t* hk = nullptr;
    uint32_t* dirty = nullptr;
    float *dv = nullptr, *da = nullptr;
    const size_t slab = (size_t)s->R * cap * s->L * sizeof(float);
    const size_t slab_old = (size_t)s->R * s->Hcap * s->L * sizeof(float);
    const size_t want = cap * 4 + (size_t)s->R * cap * 4 + slab * (s->acc ? 2 : 1);
    const size_t held = s->Hcap * 4 + (size_t)s->R * s->Hcap * 4 + slab_old * (s->acc ? 2 : 1);
    // old and new replicas exist side by side for a moment; the store's limit is judged on what stays
    if (s->dev_cap && (want > s->dev_cap || s->dev_bytes - held > s->dev_cap - want)) return NUPS_ENOMEM;
    const size_t cap_saved = s->dev_cap;
    s->dev_cap = 0;
    bool ok = nups_dev_alloc(s, (void**)&hk, cap * 4) == NUPS_OK &&
              nups_dev_alloc(s, (void**)&dirty, (size_t)s->R * cap * 4) == NUPS_OK &&
              nups_dev_alloc(s, (void**)&dv, slab) == NUPS_OK && (!s->acc || nups_dev_alloc(s, (void**)&da, slab) == NUPS_OK);
    s->dev_cap = cap_saved;
    if (!ok) {
        nups_dev_free(s, hk, cap * 4); nups_dev_free(s, dirty, (size_t)s->R * cap * 4);
        nups_dev_free(s, dv, slab); nups_dev_free(s, da, slab);
        return NUPS_ENOMEM;
    }
    // pending updates are all zero here (the caller merged them), so fresh zeroed slabs are enough
    if (s->H) CK(cudaMemcpy(hk, s->hot_keys, s->H * 4, cudaMemcpyDeviceToDevice));
    CK(cudaMemset(dirty, 0, (size_t)s->R * cap * 4));
    CK(cudaMemset(dv, 0, slab));
    if (da) CK(cudaMemset(da, 0, slab));
    CK(cudaDeviceSynchronize());
    nups_dev_free(s, s->hot_keys, s->Hcap * 4); nups_dev_free(s, s->dirty, (size_t)s->R * s->Hcap * 4);
    nups_dev_free(s, s->dval, slab_old); nups_dev_free(s, s->dacc, slab_old);
    s->hot_keys = hk; s->dirty = dirty; s->dval = dv; s->dacc = da; s->Hcap = cap;
    return NUPS_OK;
}

extern "C" nups_status nups_set_management(nups_store* s, const uint32_t* d_keys, uint64_t n, int technique, void* stream)
{
    if (!s || (n && !d_keys) || (technique != NUPS_SINGLE && technique != NUPS_REPLICATE)) return NUPS_EINVAL;
    if (n >= (1ull << 31) - 2) return NUPS_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    nups_status rc = nups_sync_internal(s, st);
    if (rc != NUPS_OK) return rc;
    CK(cudaStreamSynchronize(st));
    if (n == 0) return NUPS_OK;
    // no background merge may be enqueued or running while slots and replicas are rebuilt
    struct Bracket {
        nups_store* s;
        cudaStream_t st;
        Bracket(nups_store* s_, cudaStream_t st_) : s(s_), st(st_) { nups_background_begin(s, st); }
        ~Bracket() { nups_background_end(s, st); }
    } bracket(s, st);
    uint64_t m = technique == NUPS_REPLICATE ? n : (s->H > n ? s->H : n);
    size_t need = 2 * align256(m * 8) + align256(m * 4) + nups_scan_scratch_bytes(m) + 256;
    char* sc;
    rc = nups_scratch(s, need, &sc);
    if (rc != NUPS_OK) return rc;
    unsigned long long* flag = (unsigned long long*)sc; sc += align256(m * 8);
    unsigned long long* pos = (unsigned long long*)sc; sc += align256(m * 8);
    uint32_t* hk_new = (uint32_t*)sc; sc += align256(m * 4);
    unsigned long long* d_total = (unsigned long long*)sc; sc += 256;
    unsigned long long total = 0;
    if (technique == NUPS_REPLICATE) {
        if (s->H + n >= (1ull << 31)) return NUPS_ENOMEM;
        rc = grow_hot(s, s->H + n);
        if (rc != NUPS_OK) return rc;
        claim_kernel<<<grid_for(n, 256), 256, 0, st>>>(s->slot_of, s->num_keys, d_keys, n, s->st);
        LAUNCH_CHECK(s);
        winner_flag_kernel<<<grid_for(n, 256), 256, 0, st>>>(s->slot_of, s->num_keys, d_keys, n, flag);
        LAUNCH_CHECK(s);
        rc = nups_scan_u64(s, flag, pos, n, d_total, sc, st);
        if (rc != NUPS_OK) return rc;
        assign_slots_kernel<<<grid_for(n, 256), 256, 0, st>>>(s->slot_of, s->hot_bits, s->hot_keys, d_keys, n, flag, pos, s->H);
        LAUNCH_CHECK(s);
        CK(cudaMemcpyAsync(&total, d_total, 8, cudaMemcpyDeviceToHost, st));
        CK(cudaStreamSynchronize(st));
        s->H += total;
    } else {
        demote_kernel<<<grid_for(n, 256), 256, 0, st>>>(s->slot_of, s->hot_bits, s->num_keys, d_keys, n, s->st);
        LAUNCH_CHECK(s);
        if (s->H == 0) return NUPS_OK;
        alive_flag_kernel<<<grid_for(s->H, 256), 256, 0, st>>>(s->slot_of, s->hot_keys, s->H, flag);
        LAUNCH_CHECK(s);
        rc = nups_scan_u64(s, flag, pos, s->H, d_total, sc, st);
        if (rc != NUPS_OK) return rc;
        renumber_kernel<<<grid_for(s->H, 256), 256, 0, st>>>(s->slot_of, s->hot_keys, hk_new, s->H, flag, pos);
        LAUNCH_CHECK(s);
        CK(cudaMemcpyAsync(&total, d_total, 8, cudaMemcpyDeviceToHost, st));
        CK(cudaStreamSynchronize(st));
        if (total) CK(cudaMemcpyAsync(s->hot_keys, hk_new, total * 4, cudaMemcpyDeviceToDevice, st));
        CK(cudaStreamSynchronize(st));
        s->H = total;
    }
    return NUPS_OK;
}

extern "C" nups_status nups_get_hot(nups_store* s, uint64_t* h_n_out, uint32_t* d_keys_out, void* stream)
{
    if (!s || !h_n_out) return NUPS_EINVAL;
    *h_n_out = s->H;
    if (d_keys_out && s->H) {
        CK(cudaMemcpyAsync(d_keys_out, s->hot_keys, s->H * 4, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
        CK(cudaStreamSynchronize((cudaStream_t)stream));
    }
    return NUPS_OK;
}

// ---------------------------------------------------------------------------------------------
// ownership (the one-machine reading of "allocated at node q")
// ---------------------------------------------------------------------------------------------
__global__ void localize_request_kernel(View v, const uint32_t* __restrict__ keys, uint64_t n)
{
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const uint32_t k = keys[i];
    if (k >= v.num_keys) { flag_bad_key(v); return; }
    mark_localize(v, k, worker_of_item(i, n, v.R));
}

extern "C" nups_status nups_localize(nups_store* s, const uint32_t* d_keys, uint64_t n, void* stream)
{
    if (!s || (n && !d_keys) || n >= (1ull << 32)) return NUPS_EINVAL;
    if (!s->own || n == 0) return NUPS_OK;
    cudaStream_t st = (cudaStream_t)stream;
    nups_status rc = nups_new_epoch(s, st);
    if (rc != NUPS_OK) return rc;
    localize_request_kernel<<<grid_for(n, 256), 256, 0, st>>>(nups_view(s), d_keys, n);
    LAUNCH_CHECK(s);
    return NUPS_OK;
}

__global__ void owner_kernel(View v, const uint32_t* __restrict__ keys, uint64_t n, int* __restrict__ out)
{
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    uint32_t k = keys[i];
    int r;
    if (k >= v.num_keys) r = -1;
    else if (key_is_hot(v, k)) r = -2;
    else if (!v.own) r = -3;
    else r = (v.own[k] & 0xFFu) == NUPS_OWNER_DEFAULT ? (int)(k % v.R) : (int)(v.own[k] & 0xFFu);
    out[i] = r;
}

extern "C" nups_status nups_get_owner(nups_store* s, const uint32_t* d_keys, uint64_t n, int32_t* d_out, void* stream)
{
    if (!s || (n && (!d_keys || !d_out))) return NUPS_EINVAL;
    if (n == 0) return NUPS_OK;
    owner_kernel<<<grid_for(n, 256), 256, 0, (cudaStream_t)stream>>>(nups_view(s), d_keys, n, d_out);
    LAUNCH_CHECK(s);
    return NUPS_OK;
}

// ---------------------------------------------------------------------------------------------
// reduction-rate probe
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
red_probe_kernel(float* base, uint64_t n4)
{
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (; i < n4; i += stride) red_add_v4(base + 4 * i, zero);
}

extern "C" nups_status nups_probe_reduction_rate(nups_store* s, uint64_t bytes, uint32_t reps, double* h_gbs_out, void* stream)
{
    if (!s || !h_gbs_out || reps == 0) return NUPS_EINVAL;
    if (s->vb != 4) return NUPS_ESTATE;                       // the probe adds single-precision zeros
    cudaStream_t st = (cudaStream_t)stream;
    const uint64_t table_bytes = (uint64_t)s->num_keys * s->L * sizeof(float);
    if (bytes > table_bytes) bytes = table_bytes;
    const uint64_t n4 = bytes / 16;
    if (n4 == 0) return NUPS_EINVAL;
    cudaEvent_t a, b;
    CK(cudaEventCreate(&a));
    CK(cudaEventCreate(&b));
    const unsigned grid = grid_for(n4, 256, (unsigned)s->sm_count * 8);
    red_probe_kernel<<<grid, 256, 0, st>>>(s->val, n4);          // warm-up
    CK(cudaEventRecord(a, st));
    for (uint32_t r = 0; r < reps; ++r) red_probe_kernel<<<grid, 256, 0, st>>>(s->val, n4);
    CK(cudaEventRecord(b, st));
    s->launches += reps + 1;
    CK(cudaEventSynchronize(b));
    float ms = 0.f;
    CK(cudaEventElapsedTime(&ms, a, b));
    cudaEventDestroy(a);
    cudaEventDestroy(b);
    *h_gbs_out = (double)n4 * 16.0 * reps / (ms * 1e-3) / 1e9;
    return NUPS_OK;
}

// ---------------------------------------------------------------------------------------------
// status and statistics
// ---------------------------------------------------------------------------------------------
extern "C" nups_status nups_status_check(nups_store* s, void* stream)
{
    if (!s) return NUPS_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    int code = 0;
    CK(cudaMemcpyAsync(&code, &s->st->status, sizeof(int), cudaMemcpyDeviceToHost, st));
    CK(cudaStreamSynchronize(st));
    if (code != 0) {
        CK(cudaMemsetAsync(&s->st->status, 0, sizeof(int), st));
        CK(cudaStreamSynchronize(st));
    }
    return (nups_status)code;
}

extern "C" nups_status nups_get_stats(nups_store* s, uint64_t* h_out, void* stream)
{
    if (!s || !h_out) return NUPS_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    DevStat d;
    CK(cudaMemcpyAsync(&d, s->st, sizeof(DevStat), cudaMemcpyDeviceToHost, st));
    CK(cudaStreamSynchronize(st));
    h_out[0] = s->steps; h_out[1] = s->syncs; h_out[2] = s->launches;
    h_out[3] = d.hot_hits; h_out[4] = d.cold_hits; h_out[5] = s->H; h_out[6] = nups_background_merges(s); h_out[7] = 0;
    return NUPS_OK;
}
