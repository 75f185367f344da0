// Workload steps driving the store: skip-gram with negative sampling, ComplEx with AdaGrad and
// matrix factorization (NuPS Section 5.1).  SGNS: one warp per pair, ComplEx: one block per triple, rows
// staged in shared memory by asynchronous copies, one thread per chunk of a row; MF: one warp per cell
// with a ring of cells in flight.  Updates are pushed either straight to the store (fast mode, vector reductions) or
// into a row buffer that the ordered push applies afterwards (deterministic mode, all pulls see the
// values from before the step).
#include <mutex>
#include <type_traits>
#include <vector>

#include "nups_internal.cuh"

static inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

namespace {

__device__ __forceinline__ float clamp30(float x) { return fminf(30.f, fmaxf(-30.f, x)); }
__device__ __forceinline__ float sigmoidf_(float x) { return 1.f / (1.f + expf(-x)); }
__device__ __forceinline__ float softplusf_(float x) { return fmaxf(x, 0.f) + log1pf(expf(-fabsf(x))); }

// lane 0 of the item's warp: access count and replica/in-place statistics for one key
__device__ __forceinline__ void note_access(const View& v, uint32_t key, int slot, unsigned times)
{
    atomicAdd(v.cnt + key, (unsigned long long)times);
    atomicAdd(slot >= 0 ? &v.st->hot_hits : &v.st->cold_hits, (unsigned long long)times);
}

// offset value meaning "this key has no replica row"
constexpr unsigned long long NO_PEND = ~0ull;

// per-launch loss in fast mode: the warps of a block add their sums up in shared memory, then ONE 64-bit integer
// addition per block carries both the block's loss (fixed point, 2^-16 units, low 48 bits) and a ticket (high 16
// bits); integer additions to one address do not queue up the way floating-point ones do, need no fence and give a
// sum that does not depend on the order.  The block that draws the last ticket sees the total, writes the mean and
// clears the word.  (One addition per warp was measured: with 3,552 warps finishing together the last of them waited
// 3.5 us for its turn at that one address.)  Called once by every thread of every block, at the end of the kernel.
// Grids of the step kernels have fewer than 2^16 blocks; the sum may reach 2^32.
__device__ __forceinline__ void loss_finish(const View& v, double warp_loss, uint64_t n, float* loss_out)
{
    __shared__ double s_warp_loss[32];
    const unsigned lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    if (lane == 0) s_warp_loss[wib] = warp_loss;
    __syncthreads();
    if (threadIdx.x != 0) return;
    double block_loss = 0.0;
    for (unsigned w = 0; w < (blockDim.x + 31) / 32; ++w) block_loss += s_warp_loss[w];
    const unsigned long long nblocks = gridDim.x;
    const unsigned long long fixed = (unsigned long long)llrint(fmin(fmax(block_loss, 0.0), 4.0e9) * 65536.0);
    const unsigned long long mine = (fixed & 0xFFFFFFFFFFFFull) + (1ull << 48);
    const unsigned long long old = atomicAdd(&v.st->tmp[3], mine);
    const unsigned long long now = old + mine;
    if ((now >> 48) == nblocks) {
        if (loss_out) *loss_out = (float)((double)(now & 0xFFFFFFFFFFFFull) / 65536.0 / (double)(n ? n : 1));
        atomicExch(&v.st->tmp[3], 0ull);
    }
}

// ---------------------------------------------------------------------------------------------
// skip-gram with negative sampling.  One warp works on one pair at a time: lane l owns the float4 chunks
// l, l + 32, ... of every row (CH of them, a compile-time count, so that every shared-memory and row offset
// is an immediate).  The 2 + K stored rows of the pair are brought into shared memory by asynchronous
// 16-byte copies, all in flight at once, each lane its own column; the worker's pending replica rows of
// the replicated roles are then folded into the staged rows, so that both passes read each chunk with one
// load; the 1 + K dot products take one warp reduction each; then every lane forms and pushes its chunks
// of the updates.  Nothing is shared between the warps of a block.
// ---------------------------------------------------------------------------------------------
constexpr int SGNS_MAX_CHUNKS = 128;                               // float4 chunks of a row: at most 512 floats
// A launch over several steps adds each pair's loss (fixed point) to one of LOSS_SLOTS words of its step:
// additions to one word would queue up behind one another.
constexpr uint32_t LOSS_SLOTS = 32;
constexpr uint32_t LOSS_STEPS = 1024;                             // most steps one launch may cover; word = [slot][step]
static_assert(LOSS_SLOTS * LOSS_STEPS <= 4 * NUPS_MAX_STEP_BLOCKS, "the per-step loss words live in the loss_partial buffer");

constexpr int SGNS_WARPS = 2;                                      // warps (= pairs in flight) per block

// Gradient-norm clipping of updates to replicated keys: the bound that holds for the whole launch
// (factor x mean norm of the updates applied by finished steps; infinite before there was any).
__device__ __forceinline__ float clip_bound(const View& v)
{
    const unsigned long long cnt = v.st->clip_cnt;
    return cnt ? v.clip_factor * (float)(v.st->clip_sum / (double)cnt) : __int_as_float(0x7f800000);
}
// norm of an update as applied: cut to the bound; *scale receives the factor for the row
__device__ __forceinline__ float clip_norm(float norm, float bound, float* scale)
{
    *scale = norm > bound ? bound / norm : 1.f;
    return norm > bound ? bound : norm;
}
// fast mode: a warp's share of the running step's statistics, once per warp and launch
__device__ __forceinline__ void clip_finish(const View& v, double sum, unsigned cnt)
{
    if ((threadIdx.x & 31) == 0 && cnt) {
        atomicAdd(&v.st->clip_step_sum, sum);
        atomicAdd(&v.st->clip_step_cnt, (unsigned long long)cnt);
    }
}

// asynchronous 16-byte copy to the shared-memory address (32-bit, shared window) smem_dst
__device__ __forceinline__ void cp_async_16s(uint32_t smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}

template <bool HOT, bool DET, int KT, int CH, bool CLIP>
__global__ void __launch_bounds__(32 * SGNS_WARPS)
sgns_kernel(View v, const uint32_t* __restrict__ center, const uint32_t* __restrict__ context,
            const uint32_t* __restrict__ negs, uint64_t n, uint32_t K_arg, float lr,
            float* __restrict__ upd, uint32_t* __restrict__ ukeys, float* __restrict__ loss_item,
            float* __restrict__ loss_out, uint32_t group,
            unsigned long long* __restrict__ loss_acc, float2* __restrict__ clip_item)
{
    grid_dependency_wait();
    extern __shared__ __align__(16) float4 park_all[];
    __shared__ const float4* s_src[SGNS_WARPS][32];                // the role's stored row
    __shared__ float* s_dst[SGNS_WARPS][32];                       // where its update goes: replica row or stored row
    __shared__ float s_g[SGNS_WARPS][32];                          // d(loss)/d(score) of the role
    __shared__ float s_f[SGNS_WARPS][32];                          // clipping factor of the role's update
    constexpr uint32_t cols = 32 * CH;
    constexpr uint32_t NR = KT > 0 ? KT + 2 : 1;                   // roles kept in registers when K is fixed
    const uint32_t K = KT > 0 ? (uint32_t)KT : K_arg;
    const uint32_t lane = threadIdx.x & 31, wib = threadIdx.x >> 5, per = K + 2;
    const uint32_t L4 = v.L4;
    const uint64_t L = (uint64_t)L4 * 4;
    float4* park = park_all + (size_t)wib * per * cols + lane;          // the lane's column
    const uint32_t park_s = (uint32_t)__cvta_generic_to_shared(park);
    const uint64_t nwarps = (uint64_t)gridDim.x * SGNS_WARPS, total = n * group;
    const uint64_t w0 = (uint64_t)blockIdx.x * SGNS_WARPS + wib;
    double my_loss = 0.0;
    const float bound = CLIP ? clip_bound(v) : 0.f;
    float my_clip = 0.f;                                           // fast mode: norms applied, this lane's share
    unsigned my_clipped = 0;
    auto key_of = [&](uint64_t e) -> uint32_t {
        if (lane >= per || e >= total) return 0u;
        return lane == 0 ? context[e] : (lane <= K ? negs[e * K + lane - 1] : center[e]);
    };
    auto slot_of = [&](uint32_t key) -> int {
        return (HOT && lane < per && key < v.num_keys) ? __ldg(v.slot_of + key) : -1;
    };
    // the lookups run two pairs ahead of the work, so that neither the key nor the slot load is waited for
    uint32_t key1 = key_of(w0), key2 = key_of(w0 + nwarps);
    int slot1 = slot_of(key1);
    uint32_t step = (uint32_t)(w0 / n);
    uint64_t i = w0 - (uint64_t)step * n;
    for (uint64_t e = w0; e < total; e += nwarps, i += nwarps) {
        while (i >= n) { i -= n; ++step; }
        const uint32_t q = worker_of_item(i, n, v.R);
        const uint32_t key = key1;
        const int slot = slot1;
        key1 = key2;
        slot1 = slot_of(key2);
        key2 = key_of(e + 2 * nwarps);
        const bool ok = lane >= per || key < v.num_keys;
        if (!__all_sync(0xFFFFFFFFu, ok)) {                        // a key out of range: the whole item is skipped
            if (DET && lane < per) ukeys[i * per + lane] = NUPS_INVALID_KEY;
            if (lane == 0) { flag_bad_key(v); if (DET) loss_item[i] = 0.f; if (DET && CLIP) clip_item[i] = make_float2(0.f, 0.f); }
            continue;
        }
        const uint32_t mask = HOT ? __ballot_sync(0xFFFFFFFFu, slot >= 0) : 0u;
        __syncwarp();                                              // the previous pair's readers are done
        if (lane < per) {
            float* row = v.val + (unsigned long long)key * L;
            s_src[wib][lane] = (const float4*)row;
            s_dst[wib][lane] = slot >= 0 ? v.dval + ((unsigned long long)q * v.Hcap + (unsigned)slot) * L : row;
        }
        __syncwarp();
        float* dstp[NR];                                           // the lane's first chunk of each destination row
#pragma unroll
        for (uint32_t role = 0; role < per; ++role) {
            const float4* src = s_src[wib][role] + lane;
            float* dst = s_dst[wib][role] + 4 * lane;
            if (KT > 0) dstp[KT > 0 ? role : 0] = dst;
#pragma unroll
            for (int m = 0; m < CH; ++m)
                if (lane + 32 * m < L4) cp_async_16s(park_s + (role * cols + 32 * m) * 16, src + 32 * m);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        if (lane < per) {
            if (DET) ukeys[i * per + lane] = key;
            if (!DET && slot >= 0) mark_dirty(v, q, slot);
            if (v.count) {
                // context and centre: pulled (+ pushed in fast mode); negatives: pushed (their draw counted the sample)
                const unsigned times = (lane == 0 || lane == K + 1) ? (DET ? 1u : 2u) : (DET ? 0u : 1u);
                if (times) note_access(v, key, slot, times);
            }
            if (v.own && (lane == 0 || lane == K + 1)) mark_localize(v, key, q);
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        // fold the worker's pending replica rows (read straight from the slab) into the staged rows
        if (HOT && mask) {
#pragma unroll
            for (uint32_t role = 0; role < per; ++role) {
                if (!(mask >> role & 1u)) continue;
                const float4* pnd = (const float4*)(KT > 0 ? dstp[KT > 0 ? role : 0] : s_dst[wib][role] + 4 * lane);
#pragma unroll
                for (int m = 0; m < CH; ++m)
                    if (lane + 32 * m < L4) park[role * cols + 32 * m] = add4(park[role * cols + 32 * m], __ldg(pnd + 32 * m));
            }
        }
        // lane j ends up holding the score x_j of role j <= K
        float4 a[CH];
#pragma unroll
        for (int m = 0; m < CH; ++m)
            a[m] = lane + 32 * m < L4 ? park[(K + 1) * cols + 32 * m] : make_float4(0.f, 0.f, 0.f, 0.f);
        float x_l = 0.f;
#pragma unroll
        for (uint32_t j = 0; j <= K; ++j) {
            float d = 0.f;
#pragma unroll
            for (int m = 0; m < CH; ++m) {
                if (lane + 32 * m < L4) {
                    const float4 u = park[j * cols + 32 * m];
                    d += a[m].x * u.x + a[m].y * u.y + a[m].z * u.z + a[m].w * u.w;
                }
            }
            d = warp_sum(d);
            if (lane == j) x_l = d;
        }
        x_l = clamp30(x_l);
        const float g_l = sigmoidf_(x_l) - (lane == 0 ? 1.f : 0.f);
        float gk[NR];
        if (KT > 0) {
#pragma unroll
            for (int j = 0; j <= KT; ++j) gk[j] = __shfl_sync(0xFFFFFFFFu, g_l, j);
        } else {
            s_g[wib][lane] = g_l;
        }
        float loss_l = lane == 0 ? softplusf_(-x_l) : (lane <= K ? softplusf_(x_l) : 0.f);
        loss_l = warp_sum(loss_l);
        // clipping: the update of role j <= K is -lr g_j a, of norm lr |g_j| |a|; lane j holds its factor
        float f_l = 1.f, clip_sum_item = 0.f;
        const bool clip_here = CLIP && mask != 0u;                 // some role of the pair is replicated
        if (clip_here) {
            float a2 = 0.f;
#pragma unroll
            for (int m = 0; m < CH; ++m) a2 += a[m].x * a[m].x + a[m].y * a[m].y + a[m].z * a[m].z + a[m].w * a[m].w;
            const float an = sqrtf(warp_sum(a2));
            float applied = 0.f;
            if (lane <= K && (mask >> lane & 1u)) applied = clip_norm(lr * fabsf(g_l) * an, bound, &f_l);
            if (DET) clip_sum_item = warp_sum(applied);            // per item, in a fixed order
            else my_clip += applied;                               // summed over the lanes when the kernel ends
        }
        float fk[NR];
        if (CLIP && KT > 0) {
#pragma unroll
            for (int j = 0; j <= KT; ++j) fk[j] = __shfl_sync(0xFFFFFFFFu, f_l, j);
        } else if (CLIP) {
            s_f[wib][lane] = f_l;
        }
        __syncwarp();
        float4 gvv[CLIP ? CH : 1];
#pragma unroll
        for (int m = 0; m < CH; ++m) {
            if (lane + 32 * m >= L4) { if (CLIP) gvv[CLIP ? m : 0] = make_float4(0.f, 0.f, 0.f, 0.f); continue; }
            float4 gv = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (uint32_t j = 0; j <= K; ++j) {
                const float g = KT > 0 ? gk[KT > 0 ? j : 0] : s_g[wib][j];
                const float4 u = park[j * cols + 32 * m];
                float sc = -lr * g;
                if (CLIP) sc *= KT > 0 ? fk[KT > 0 ? j : 0] : s_f[wib][j];
                const float4 du = make_float4(sc * a[m].x, sc * a[m].y, sc * a[m].z, sc * a[m].w);
                if (DET) ((float4*)(upd + (i * per + j) * L))[lane + 32 * m] = du;
                else red_add_v4((KT > 0 ? dstp[KT > 0 ? j : 0] : s_dst[wib][j] + 4 * lane) + 128 * m, du);
                gv.x += g * u.x; gv.y += g * u.y; gv.z += g * u.z; gv.w += g * u.w;
            }
            if (CLIP) { gvv[CLIP ? m : 0] = gv; continue; }          // the centre's update waits for its norm
            const float4 dv = make_float4(-lr * gv.x, -lr * gv.y, -lr * gv.z, -lr * gv.w);
            if (DET) ((float4*)(upd + (i * per + K + 1) * L))[lane + 32 * m] = dv;
            else red_add_v4((KT > 0 ? dstp[KT > 0 ? KT + 1 : 0] : s_dst[wib][K + 1] + 4 * lane) + 128 * m, dv);
        }
        if (CLIP) {
            float fc = 1.f;
            if (mask >> (K + 1) & 1u) {                            // the centre word is replicated
                float g2 = 0.f;
#pragma unroll
                for (int m = 0; m < CH; ++m) {
                    const float4 gv = gvv[CLIP ? m : 0];
                    g2 += gv.x * gv.x + gv.y * gv.y + gv.z * gv.z + gv.w * gv.w;
                }
                const float applied = clip_norm(lr * sqrtf(warp_sum(g2)), bound, &fc);
                if (DET) clip_sum_item += applied;
                else if (lane == 0) my_clip += applied;
            }
            const float sc = -lr * fc;
#pragma unroll
            for (int m = 0; m < CH; ++m) {
                if (lane + 32 * m >= L4) continue;
                const float4 gv = gvv[CLIP ? m : 0];
                const float4 dv = make_float4(sc * gv.x, sc * gv.y, sc * gv.z, sc * gv.w);
                if (DET) ((float4*)(upd + (i * per + K + 1) * L))[lane + 32 * m] = dv;
                else red_add_v4((KT > 0 ? dstp[KT > 0 ? KT + 1 : 0] : s_dst[wib][K + 1] + 4 * lane) + 128 * m, dv);
            }
            if (DET) { if (lane == 0) clip_item[i] = make_float2(clip_sum_item, (float)__popc(mask)); }
            else my_clipped += __popc(mask);
        }
        if (lane == 0) {
            if (DET) loss_item[i] = loss_l;
            if (loss_acc) atomicAdd(loss_acc + (uint32_t)(w0 % LOSS_SLOTS) * LOSS_STEPS + step, (unsigned long long)llrintf(fminf(loss_l, 60000.f) * 65536.f));
            else my_loss += (double)loss_l;
        }
    }
    if (!DET && !loss_acc) loss_finish(v, my_loss, n, loss_out);
    if (CLIP && !DET) clip_finish(v, (double)warp_sum(my_clip), my_clipped);
}

// ---------------------------------------------------------------------------------------------
// skip-gram, fast mode with three negatives per pair: rows in registers, runs of one centre word summed.
// A warp takes a stretch of consecutive pairs of the launch.  Pairs arrive centre by centre (a position of
// the token stream is paired with every position of its window in turn), so the centre word stays the same
// over a run of pairs: its row is read once per run and kept in registers, the updates that the run's pairs
// make to it are summed in registers and added once when the run ends.  All pairs of a run therefore see the
// centre's row from before the run, which is what the batch semantics of the deterministic mode gives every
// pair of a step; the rows of context words and negatives are read and updated pair by pair as before.
// The four other rows of a pair go straight from global memory into registers (lane l owns the 16-byte chunks
// l, l + 32, ...), the four scores are reduced together (6 shuffles instead of 20), every lane then forms its
// chunks of the updates.  Keys and replica slots are looked up 32 pairs at a time, one pair per lane.
// ---------------------------------------------------------------------------------------------
constexpr int SGNS_RUN_THREADS = 128;
constexpr int SGNS_RUN_BLOCKS = 4;         // resident blocks per multiprocessor: 128 registers a thread (3 blocks at 158: 103 vs 95 us per launch)

template <bool HOT, int CH>
__global__ void __launch_bounds__(SGNS_RUN_THREADS, SGNS_RUN_BLOCKS)
sgns_runs_kernel(View v, const uint32_t* __restrict__ center, const uint32_t* __restrict__ context,
                 const uint32_t* __restrict__ negs, uint64_t n, float lr, float* __restrict__ loss_out, uint32_t group,
                 unsigned long long* __restrict__ loss_acc)
{
    grid_dependency_wait();
    constexpr unsigned FULL = 0xFFFFFFFFu;
    constexpr int K = 3;
    const unsigned lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t nwarps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    const uint32_t L4 = v.L4;
    const uint64_t total = n * group;
    const uint64_t stretch = (total + nwarps - 1) / nwarps;
    const uint64_t first = warp * stretch < total ? warp * stretch : total;
    const uint64_t last = first + stretch < total ? first + stretch : total;          // this warp's pairs: [first, last)
    const float4* val4 = reinterpret_cast<const float4*>(v.val);
    const float4* slab4 = reinterpret_cast<const float4*>(v.dval);

    // one window = 32 consecutive pairs, lane l holds pair l: keys of the five roles (all invalid when one is) and slots
    struct Window { uint32_t k[K + 2]; int s[K + 2]; };                              // roles: context, negatives, centre
    auto load_window = [&](uint64_t base) {
        Window w;
#pragma unroll
        for (int r = 0; r < K + 2; ++r) { w.k[r] = NUPS_INVALID_KEY; w.s[r] = -1; }
        const uint64_t e = base + lane;
        if (e < last) {
            uint32_t k[K + 2];
            k[0] = context[e];
#pragma unroll
            for (int j = 0; j < K; ++j) k[1 + j] = negs[e * K + j];
            k[K + 1] = center[e];
            bool ok = true;
#pragma unroll
            for (int r = 0; r < K + 2; ++r) ok = ok && k[r] < v.num_keys;
            if (ok) {
#pragma unroll
                for (int r = 0; r < K + 2; ++r) { w.k[r] = k[r]; if (HOT) { const int sl = __ldg(v.slot_of + k[r]); w.s[r] = sl < 0 ? -1 : sl; } }
            } else {
                flag_bad_key(v);
            }
        }
        return w;
    };
    auto fetch_row = [&](float4 (&dst)[CH], const float4* row) {
#pragma unroll
        for (int m = 0; m < CH; ++m) {
            const uint32_t c = lane + 32 * m;
            dst[m] = c < L4 ? __ldg(row + c) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    auto fold_pending = [&](float4 (&dst)[CH], const float4* pend) {
#pragma unroll
        for (int m = 0; m < CH; ++m) {
            const uint32_t c = lane + 32 * m;
            if (c < L4) dst[m] = add4(dst[m], pend[c]);
        }
    };

    Window cur = load_window(first), nxt = load_window(first + 32);
    float4 a[CH], held[CH];                                 // the run's centre row; the summed updates to it
    float* held_dst = nullptr;                              // where they go: replica row or stored row
    auto flush_held = [&]() {
        if (!held_dst) return;
#pragma unroll
        for (int m = 0; m < CH; ++m) {
            const uint32_t c = lane + 32 * m;
            if (c < L4) red_add_v4(held_dst + 4 * c, held[m]);
        }
        held_dst = nullptr;
    };
    // item index within its step, its worker and the worker's last item, kept up as the pairs go by
    uint32_t step = (uint32_t)((first < total ? first : 0) / n);
    uint64_t i = (first < total ? first : 0) - (uint64_t)step * n;
    uint32_t q = worker_of_item(i, n, v.R);
    uint64_t q_end = worker_first_item(q + 1, n, v.R);
    float step_loss = 0.f;                                  // this lane's share of the running step's loss
    double my_loss = 0.0;
    auto close_step = [&]() {
        const float sum = warp_sum(step_loss);
        step_loss = 0.f;
        if (loss_acc) {
            if (lane == 0 && sum != 0.f)
                atomicAdd(loss_acc + (uint32_t)(warp % LOSS_SLOTS) * LOSS_STEPS + step,
                          (unsigned long long)llrintf(fminf(sum, 4.0e9f / 65536.f) * 65536.f));
        } else {
            my_loss += (double)sum;
        }
    };
    for (uint64_t base = first; base < last; base += 32) {
        const uint32_t in_window = (uint32_t)min((uint64_t)32, last - base);
        for (uint32_t t = 0; t < in_window; ++t, ++i) {
            if (i >= n) { close_step(); i -= n; ++step; q = 0; q_end = worker_first_item(1, n, v.R); }
            while (i >= q_end) q_end = worker_first_item(++q + 1, n, v.R);
            uint32_t key[K + 2];
            int slot[K + 2];
#pragma unroll
            for (int r = 0; r < K + 2; ++r) {
                key[r] = __shfl_sync(FULL, cur.k[r], t);
                slot[r] = HOT ? __shfl_sync(FULL, cur.s[r], t) : -1;
            }
            if (key[K + 1] == NUPS_INVALID_KEY) continue;                      // a key out of range: flagged at the lookup
            // destination rows: the worker's replica row of a replicated key, else the stored row
            float* dst[K + 2];
#pragma unroll
            for (int r = 0; r < K + 2; ++r)
                dst[r] = slot[r] >= 0 ? v.dval + ((uint64_t)q * v.Hcap + (unsigned)slot[r]) * L4 * 4
                                      : v.val + (uint64_t)key[r] * L4 * 4;
            float4 u[K + 1][CH];
#pragma unroll
            for (int j = 0; j <= K; ++j) fetch_row(u[j], val4 + (uint64_t)key[j] * L4);
            if (dst[K + 1] != held_dst) {                                        // a new run: another centre word or worker
                flush_held();
                fetch_row(a, val4 + (uint64_t)key[K + 1] * L4);
                if (HOT && slot[K + 1] >= 0) fold_pending(a, reinterpret_cast<const float4*>(dst[K + 1]));
#pragma unroll
                for (int m = 0; m < CH; ++m) held[m] = make_float4(0.f, 0.f, 0.f, 0.f);
                held_dst = dst[K + 1];
                if (HOT && slot[K + 1] >= 0 && lane == 0) mark_dirty(v, q, slot[K + 1]);
            }
            if (HOT) {
#pragma unroll
                for (int j = 0; j <= K; ++j)
                    if (slot[j] >= 0) fold_pending(u[j], reinterpret_cast<const float4*>(dst[j]));
            }
            if (HOT && lane == 0) {
#pragma unroll
                for (int j = 0; j <= K; ++j)
                    if (slot[j] >= 0) mark_dirty(v, q, slot[j]);
            }
            // the four scores at once: after the halving steps lane l holds score 2 * bit4(l) + bit3(l)
            float x[K + 1];
#pragma unroll
            for (int j = 0; j <= K; ++j) {
                float d = 0.f;
#pragma unroll
                for (int m = 0; m < CH; ++m) d += a[m].x * u[j][m].x + a[m].y * u[j][m].y + a[m].z * u[j][m].z + a[m].w * u[j][m].w;
                x[j] = d;
            }
            {
                const bool up16 = (lane & 16) != 0, up8 = (lane & 8) != 0;
                const float k0 = (up16 ? x[2] : x[0]) + __shfl_xor_sync(FULL, up16 ? x[0] : x[2], 16);
                const float k1 = (up16 ? x[3] : x[1]) + __shfl_xor_sync(FULL, up16 ? x[1] : x[3], 16);
                float y = (up8 ? k1 : k0) + __shfl_xor_sync(FULL, up8 ? k0 : k1, 8);
                y += __shfl_xor_sync(FULL, y, 4);
                y += __shfl_xor_sync(FULL, y, 2);
                y += __shfl_xor_sync(FULL, y, 1);
                const uint32_t mine = ((lane >> 4) & 1u) * 2 + ((lane >> 3) & 1u);      // the score this lane holds
                y = clamp30(y);
                const float g_l = sigmoidf_(y) - (mine == 0 ? 1.f : 0.f);
                if ((lane & 7u) == 0) step_loss += mine == 0 ? softplusf_(-y) : softplusf_(y);
#pragma unroll
                for (int j = 0; j <= K; ++j) x[j] = __shfl_sync(FULL, g_l, 16 * (j >> 1) + 8 * (j & 1));   // x[j] = g_j now
            }
#pragma unroll
            for (int m = 0; m < CH; ++m) {
                const uint32_t c = lane + 32 * m;
                if (c >= L4) continue;
                float4 gv = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int j = 0; j <= K; ++j) {
                    const float sc = -lr * x[j];
                    red_add_v4(dst[j] + 4 * c, make_float4(sc * a[m].x, sc * a[m].y, sc * a[m].z, sc * a[m].w));
                    gv.x += x[j] * u[j][m].x; gv.y += x[j] * u[j][m].y; gv.z += x[j] * u[j][m].z; gv.w += x[j] * u[j][m].w;
                }
                held[m].x += -lr * gv.x; held[m].y += -lr * gv.y; held[m].z += -lr * gv.z; held[m].w += -lr * gv.w;
            }
        }
        cur = nxt;
        nxt = load_window(base + 64);
    }
    flush_held();
    close_step();
    if (!loss_acc) loss_finish(v, my_loss, n, loss_out);
}

// ---------------------------------------------------------------------------------------------
// ComplEx with AdaGrad.  Rows are [re(0..d-1) | im(0..d-1)], d = L/2 (even).  One block of 128 threads
// works on one triple at a time.  All 2 * (3 + K) rows of the triple (values and accumulators) are brought
// into shared memory as they lie in memory, by asynchronous 16-byte copies that are all in flight at once
// (thread t moves chunk t of every row and folds the worker's pending replica updates into what it moved).
// For the arithmetic thread c owns the two adjacent complex components 2c, 2c+1 (a float2 of the real half
// and the matching float2 of the imaginary half), so d <= 256.  Pass 1 forms the thread's part of the
// 1 + K scores; they are added up across the block together (one transposed warp reduction for up to 16
// scores instead of one reduction per score).  Pass 2 forms the gradients and leaves every role's AdaGrad
// update in the shared-memory rows it no longer needs; after a barrier thread t hands chunk t of every
// update row to the store with one 128-bit reduction (fast mode) or one 128-bit store into the row buffer
// of the ordered push (deterministic mode).
// Deterministic mode computes in double precision between pull and push (scores, gradients, AdaGrad step),
// rounding once when the update rows are stored; fast mode computes in single precision.
// ---------------------------------------------------------------------------------------------
constexpr int CPX_THREADS = 128;
constexpr int CPX_MAX_KEYS = 34;          // 3 + K with K <= 30, rounded up
constexpr int CPX_NS = 16;                // up to this many scores are reduced together
// the 16-byte chunks of a row that thread tid moves: one (rows of up to 512 fp32 values), two with 8-byte values
#define NUPS_CPX_CHUNKS(c) _Pragma("unroll") for (uint32_t c = tid; c < L4 && c < (F64 ? 2u : 1u) * CPX_THREADS; c += CPX_THREADS)

template <class T> struct CX { T re[2], im[2]; };

template <class T> __device__ __forceinline__ CX<T> cx_zero() { CX<T> z; z.re[0] = z.re[1] = z.im[0] = z.im[1] = T(0); return z; }

__device__ __forceinline__ float mul_rn(float a, float b) { return __fmul_rn(a, b); }
__device__ __forceinline__ double mul_rn(double a, double b) { return __dmul_rn(a, b); }
__device__ __forceinline__ float sub_rn(float a, float b) { return __fsub_rn(a, b); }
__device__ __forceinline__ double sub_rn(double a, double b) { return __dsub_rn(a, b); }

// the thread's components of a row staged in shared memory (S = the table's value type, T = the type computed in):
// two adjacent values of the real half and the two matching ones of the imaginary half, each pair one vector access
// (d is even, so both pairs are aligned to their own size)
template <class T>
__device__ __forceinline__ CX<T> cx_load(const float* row, uint32_t d, uint32_t c)
{
    const float2 a = *reinterpret_cast<const float2*>(row + 2 * c);
    const float2 b = *reinterpret_cast<const float2*>(row + d + 2 * c);
    CX<T> x;
    x.re[0] = (T)a.x; x.re[1] = (T)a.y; x.im[0] = (T)b.x; x.im[1] = (T)b.y;
    return x;
}
template <class T>
__device__ __forceinline__ CX<T> cx_load(const double* row, uint32_t d, uint32_t c)
{
    const double2 a = *reinterpret_cast<const double2*>(row + 2 * c);
    const double2 b = *reinterpret_cast<const double2*>(row + d + 2 * c);
    CX<T> x;
    x.re[0] = (T)a.x; x.re[1] = (T)a.y; x.im[0] = (T)b.x; x.im[1] = (T)b.y;
    return x;
}
__device__ __forceinline__ void cx_store(float* row, uint32_t d, uint32_t c, float r0, float r1, float i0, float i1)
{
    *reinterpret_cast<float2*>(row + 2 * c) = make_float2(r0, r1);
    *reinterpret_cast<float2*>(row + d + 2 * c) = make_float2(i0, i1);
}
__device__ __forceinline__ void cx_store(double* row, uint32_t d, uint32_t c, double r0, double r1, double i0, double i1)
{
    *reinterpret_cast<double2*>(row + 2 * c) = make_double2(r0, r1);
    *reinterpret_cast<double2*>(row + d + 2 * c) = make_double2(i0, i1);
}

template <class T>
__device__ __forceinline__ T cx_score(const CX<T>& h, const CX<T>& r, const CX<T>& t)
{
    T s = T(0);
#pragma unroll
    for (int k = 0; k < 2; ++k)
        s += h.re[k] * r.re[k] * t.re[k] + h.im[k] * r.re[k] * t.im[k] + h.re[k] * r.im[k] * t.im[k] - h.im[k] * r.im[k] * t.re[k];
    return s;
}

// g_h += coef * d(phi)/d(h), likewise for r and t (any of the three may be skipped).  Differences of
// products are formed without fused multiply-add, so that a gradient that cancels exactly
// (head == tail) is exactly zero here too.
template <class T>
__device__ __forceinline__ void cx_grads(const CX<T>& h, const CX<T>& r, const CX<T>& t, T coef, CX<T>* gh, CX<T>* gr, CX<T>* gt)
{
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const T hr = h.re[k], hi = h.im[k], rr = r.re[k], ri = r.im[k], tr = t.re[k], ti = t.im[k];
        if (gh) { gh->re[k] += coef * (rr * tr + ri * ti); gh->im[k] += coef * sub_rn(mul_rn(rr, ti), mul_rn(ri, tr)); }
        if (gt) { gt->re[k] += coef * sub_rn(mul_rn(hr, rr), mul_rn(hi, ri)); gt->im[k] += coef * (hi * rr + hr * ri); }
        if (gr) { gr->re[k] += coef * (hr * tr + hi * ti); gr->im[k] += coef * sub_rn(mul_rn(hr, ti), mul_rn(hi, tr)); }
    }
}

// step = -lr * g / (sqrt(a + g^2) + eps).  Single precision (fast mode): the hardware's reciprocal square
// root and approximate division (2 ulp each).  Double precision (deterministic mode): IEEE sqrt and division.
__device__ __forceinline__ float adagrad_step(float g, float g2, float a, float lr, float eps)
{
    const float y = a + g2;
    const float root = y > 0.f ? y * rsqrtf(y) : 0.f;
    return __fdividef(-lr * g, root + eps);
}
__device__ __forceinline__ double adagrad_step(double g, double g2, double a, double lr, double eps)
{
    return -lr * g / (sqrt(a + g2) + eps);
}

// AdaGrad update of one key role from the thread's part of its summed gradient: the update rows
// (value: -lr g / (sqrt(acc_pulled + g^2) + eps), accumulator: g^2) replace the role's staged rows
template <class T, class S>
__device__ __forceinline__ void cx_adagrad(const CX<T>& g, S* val_row, S* acc_row, uint32_t d, uint32_t c, T lr, T eps)
{
    const CX<T> a = cx_load<T>(acc_row, d, c);
    const T r0 = g.re[0] * g.re[0], r1 = g.re[1] * g.re[1], i0 = g.im[0] * g.im[0], i1 = g.im[1] * g.im[1];
    cx_store(val_row, d, c, (S)adagrad_step(g.re[0], r0, a.re[0], lr, eps), (S)adagrad_step(g.re[1], r1, a.re[1], lr, eps),
                (S)adagrad_step(g.im[0], i0, a.im[0], lr, eps), (S)adagrad_step(g.im[1], i1, a.im[1], lr, eps));
    cx_store(acc_row, d, c, (S)r0, (S)r1, (S)i0, (S)i1);
}

template <class T>
__device__ __forceinline__ T warp_sum_t(T x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
    return x;
}

// Sixteen sums over the warp at once: every lane brings v[0..15]; every lane returns the warp's total of
// entry (lane >> 1) & 15.  Each step halves what a lane holds: the lane keeps the half its bit selects and
// hands the other half to its partner (8 + 4 + 2 + 1 shuffles, one more for the last pair of lanes).
template <class T>
__device__ __forceinline__ T warp_sum16(T (&v)[CPX_NS], unsigned lane)
{
#pragma unroll
    for (int half = CPX_NS / 2, bit = 16; half >= 1; half >>= 1, bit >>= 1) {
        const bool upper = (lane & bit) != 0;
#pragma unroll
        for (int k = 0; k < half; ++k) {
            const T send = upper ? v[k] : v[k + half];
            const T keep = upper ? v[k + half] : v[k];
            v[k] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, bit);
        }
    }
    return v[0] + __shfl_xor_sync(0xFFFFFFFFu, v[0], 1);
}

__device__ __forceinline__ float clampT(float x) { return clamp30(x); }
__device__ __forceinline__ double clampT(double x) { return fmin(30.0, fmax(-30.0, x)); }
__device__ __forceinline__ float sigmoidT(float x) { return sigmoidf_(x); }
__device__ __forceinline__ double sigmoidT(double x) { return 1.0 / (1.0 + exp(-x)); }
__device__ __forceinline__ float softplusT(float x) { return softplusf_(x); }
__device__ __forceinline__ double softplusT(double x) { return fmax(x, 0.0) + log1p(exp(-fabs(x))); }

template <bool HOT, bool DET, bool RED16, bool F64>
__global__ void __launch_bounds__(CPX_THREADS, F64 ? 2 : 4)
complex_kernel(View v, const uint32_t* __restrict__ hk, const uint32_t* __restrict__ rk, const uint32_t* __restrict__ tk,
               const uint32_t* __restrict__ negs, uint64_t n, uint32_t K, float lr, float eps, float* __restrict__ uval,
               float* __restrict__ uacc, uint32_t* __restrict__ ukeys, float* __restrict__ loss_item,
               float* __restrict__ loss_out)
{
    grid_dependency_wait();
    using S = typename std::conditional<F64, double, float>::type;          // what the tables hold
    using T = typename std::conditional<DET || F64, double, float>::type;   // what the step computes in
    // rows[2 * role] = the role's value row, rows[2 * role + 1] = its accumulator row, as they lie in memory
    extern __shared__ __align__(16) unsigned char rows_raw[];
    S* rows = reinterpret_cast<S*>(rows_raw);
    __shared__ unsigned long long s_row[CPX_MAX_KEYS], s_pend[CPX_MAX_KEYS];   // offsets in 4-byte units
    __shared__ T s_part[CPX_THREADS / 32][32];                     // per-warp sums of the scores
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t L4 = v.L4, per = K + 3;                         // 16-byte chunks of a row
    const uint32_t L = F64 ? L4 * 2 : L4 * 4, d = L / 2;           // values per row, complex components
    const uint32_t LU = L4 * 4;                                    // row length in 4-byte units
    const bool mine = tid < d / 2;                                 // threads beyond the row width only help reduce
    const T lrT = (T)lr, epsT = (T)eps;
    double my_loss = 0.0;
    s_part[warp][lane] = T(0);
    for (uint64_t i = blockIdx.x; i < n; i += gridDim.x) {
        const uint32_t q = worker_of_item(i, n, v.R);
        // thread j < 3 + K looks up role j: head, relation, tail, negatives
        uint32_t key = 0;
        if (tid < per) key = tid == 0 ? hk[i] : tid == 1 ? rk[i] : tid == 2 ? tk[i] : negs[i * K + tid - 3];
        // one decision for the whole block (the barrier also ends the previous triple's use of the rows)
        const int ok = __syncthreads_and(tid >= per || key < v.num_keys);
        if (!ok) {                                                 // a key out of range: the whole item is skipped
            if (DET && tid < per) ukeys[i * per + tid] = NUPS_INVALID_KEY;
            if (tid == 0) { flag_bad_key(v); if (DET) loss_item[i] = 0.f; }
            continue;
        }
        if (tid < per) {
            int slot = HOT ? __ldg(v.slot_of + key) : -1;
            if (slot < 0) slot = -1;
            s_row[tid] = (unsigned long long)key * LU;
            s_pend[tid] = slot >= 0 ? ((unsigned long long)q * v.Hcap + (unsigned)slot) * LU : NO_PEND;
            if (DET) ukeys[i * per + tid] = key;
            if (!DET && slot >= 0) mark_dirty(v, q, slot);
            if (v.count) {
                const unsigned times = (tid < 3 ? 1u : 0u) + (DET ? 0u : 1u);       // pulled (+ pushed in fast mode)
                if (times) note_access(v, key, slot, times);
            }
            if (v.own && tid < 3) mark_localize(v, key, q);
        }
        __syncthreads();
        if constexpr (!F64) {                                      // at most one chunk per thread
            if (tid < L4) {
                const uint32_t dst = (uint32_t)__cvta_generic_to_shared(rows) + 16 * tid;
                for (uint32_t role = 0; role < per; ++role) {
                    cp_async_16s(dst + (2 * role) * LU * 4, v.val + s_row[role] + 4 * tid);
                    cp_async_16s(dst + (2 * role + 1) * LU * 4, v.acc + s_row[role] + 4 * tid);
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
            }
        } else {
            const uint32_t dst = (uint32_t)__cvta_generic_to_shared(rows);
            for (uint32_t role = 0; role < per; ++role) {
                NUPS_CPX_CHUNKS(c) {
                    cp_async_16s(dst + ((2 * role) * L4 + c) * 16, v.val + s_row[role] + 4 * c);
                    cp_async_16s(dst + ((2 * role + 1) * L4 + c) * 16, v.acc + s_row[role] + 4 * c);
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        // while this triple is worked on, the rows of the block's next triple start moving towards L2
        {
            const uint64_t nx = i + gridDim.x;
            if (nx < n) {
                const uint32_t lines_per_row = (LU * 4 + 127) / 128;
                for (uint32_t e = tid; e < per * lines_per_row; e += CPX_THREADS) {
                    const uint32_t role = e / lines_per_row, line = e % lines_per_row;
                    const uint32_t k = role == 0 ? hk[nx] : role == 1 ? rk[nx] : role == 2 ? tk[nx] : negs[nx * K + role - 3];
                    const size_t off = (size_t)k * LU + (size_t)line * 32;
                    if (k < v.num_keys && off + 32 <= (size_t)v.num_keys * LU) {      // a whole line inside the table
                        prefetch_l2(v.val + off);
                        prefetch_l2(v.acc + off);
                    }
                }
            }
        }
        if constexpr (!F64) {
            if (tid < L4) {
                asm volatile("cp.async.wait_group 0;" ::: "memory");
                if (HOT) {
                    // the worker's pending replica updates join the chunks this thread staged
                    for (uint32_t role = 0; role < per; ++role) {
                        const unsigned long long pend = s_pend[role];
                        if (pend == NO_PEND) continue;
                        float4* pv = reinterpret_cast<float4*>(rows + (size_t)(2 * role) * L) + tid;
                        float4* pa = reinterpret_cast<float4*>(rows + (size_t)(2 * role + 1) * L) + tid;
                        *pv = add4(*pv, *(reinterpret_cast<const float4*>(v.dval + pend) + tid));
                        *pa = add4(*pa, *(reinterpret_cast<const float4*>(v.dacc + pend) + tid));
                    }
                }
            }
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            if (HOT) {
                float4* staged = reinterpret_cast<float4*>(rows_raw);
                for (uint32_t role = 0; role < per; ++role) {
                    const unsigned long long pend = s_pend[role];
                    if (pend == NO_PEND) continue;
                    NUPS_CPX_CHUNKS(c) {
                        float4* pv = staged + (size_t)(2 * role) * L4 + c;
                        float4* pa = staged + (size_t)(2 * role + 1) * L4 + c;
                        *pv = add_chunk<true>(*pv, *(reinterpret_cast<const float4*>(v.dval + pend) + c));
                        *pa = add_chunk<true>(*pa, *(reinterpret_cast<const float4*>(v.dacc + pend) + c));
                    }
                }
            }
        }
        __syncthreads();
        auto val_row = [&](uint32_t role) { return rows + (size_t)(2 * role) * L; };
        auto acc_row = [&](uint32_t role) { return rows + (size_t)(2 * role + 1) * L; };
        CX<T> h = cx_zero<T>(), r = cx_zero<T>(), t = cx_zero<T>();
        if (mine) { h = cx_load<T>(val_row(0), d, tid); r = cx_load<T>(val_row(1), d, tid); t = cx_load<T>(val_row(2), d, tid); }
        // pass 1: the thread's part of every score; lane j < 32 of each warp ends up with the warp's sum of score j
        if (RED16) {
            T sc[CPX_NS];
            sc[0] = mine ? cx_score(h, r, t) : T(0);
#pragma unroll
            for (int j = 0; j < CPX_NS - 1; ++j) {
                sc[j + 1] = T(0);
                if ((uint32_t)j < K && mine) {
                    const CX<T> e = cx_load<T>(val_row(3 + j), d, tid);
                    sc[j + 1] = (j & 1) == 0 ? cx_score(e, r, t) : cx_score(h, r, e);
                }
            }
            const T tot = warp_sum16(sc, lane);
            if ((lane & 1u) == 0) s_part[warp][lane >> 1] = tot;
        } else {
            T part = T(0);
            {
                const T sc = warp_sum_t(mine ? cx_score(h, r, t) : T(0));
                if (lane == 0) part = sc;
            }
            for (uint32_t j = 0; j < K; ++j) {
                T sc = T(0);
                if (mine) {
                    const CX<T> e = cx_load<T>(val_row(3 + j), d, tid);
                    sc = (j & 1) == 0 ? cx_score(e, r, t) : cx_score(h, r, e);
                }
                sc = warp_sum_t(sc);
                if (lane == j + 1) part = sc;
            }
            s_part[warp][lane] = part;
        }
        __syncthreads();
        // every thread needs every score: lane j adds the warps' sums of score j, then they are passed around
        T phi_l = T(0);
#pragma unroll
        for (int w = 0; w < CPX_THREADS / 32; ++w) phi_l += s_part[w][lane];
        phi_l = clampT(phi_l);
        const T coef_l = lane == 0 ? sigmoidT(phi_l) - T(1) : sigmoidT(phi_l);
        T loss_l = lane == 0 ? softplusT(-phi_l) : (lane <= K ? softplusT(phi_l) : T(0));
        loss_l = warp_sum_t(loss_l);
        // pass 2: gradients; each role's update rows replace its staged rows
        CX<T> gh = cx_zero<T>(), gr = cx_zero<T>(), gt = cx_zero<T>();
        cx_grads(h, r, t, __shfl_sync(0xFFFFFFFFu, coef_l, 0), &gh, &gr, &gt);
        for (uint32_t j = 0; j < K; ++j) {
            const T coef = __shfl_sync(0xFFFFFFFFu, coef_l, j + 1);
            if (!mine) continue;
            const CX<T> e = cx_load<T>(val_row(3 + j), d, tid);
            CX<T> ge = cx_zero<T>();
            if ((j & 1) == 0) cx_grads(e, r, t, coef, &ge, &gr, &gt);
            else cx_grads(h, r, e, coef, &gh, &gr, &ge);
            cx_adagrad(ge, val_row(3 + j), acc_row(3 + j), d, tid, lrT, epsT);
        }
        if (mine) {
            cx_adagrad(gh, val_row(0), acc_row(0), d, tid, lrT, epsT);
            cx_adagrad(gr, val_row(1), acc_row(1), d, tid, lrT, epsT);
            cx_adagrad(gt, val_row(2), acc_row(2), d, tid, lrT, epsT);
        }
        __syncthreads();
        if constexpr (!F64) {
            if (tid < L4) {
                for (uint32_t role = 0; role < per; ++role) {
                    const float4 dv = reinterpret_cast<const float4*>(val_row(role))[tid];
                    const float4 da = reinterpret_cast<const float4*>(acc_row(role))[tid];
                    if (DET) {
                        reinterpret_cast<float4*>(uval + (i * per + role) * (uint64_t)LU)[tid] = dv;
                        reinterpret_cast<float4*>(uacc + (i * per + role) * (uint64_t)LU)[tid] = da;
                    } else {
                        const unsigned long long pend = s_pend[role];
                        float* ov = pend != NO_PEND ? v.dval + pend : v.val + s_row[role];
                        float* oa = pend != NO_PEND ? v.dacc + pend : v.acc + s_row[role];
                        red_add_v4(ov + 4 * tid, dv);
                        red_add_v4(oa + 4 * tid, da);
                    }
                }
            }
        } else {
            for (uint32_t role = 0; role < per; ++role) {
                NUPS_CPX_CHUNKS(c) {
                    const float4 dv = reinterpret_cast<const float4*>(val_row(role))[c];
                    const float4 da = reinterpret_cast<const float4*>(acc_row(role))[c];
                    if (DET) {
                        reinterpret_cast<float4*>(uval + (i * per + role) * (uint64_t)LU)[c] = dv;
                        reinterpret_cast<float4*>(uacc + (i * per + role) * (uint64_t)LU)[c] = da;
                    } else {
                        const unsigned long long pend = s_pend[role];
                        float* ov = pend != NO_PEND ? v.dval + pend : v.val + s_row[role];
                        float* oa = pend != NO_PEND ? v.dacc + pend : v.acc + s_row[role];
                        red_add_chunk<true>(ov + 4 * c, dv);
                        red_add_chunk<true>(oa + 4 * c, da);
                    }
                }
            }
        }
        if (tid == 0) {
            if (DET) loss_item[i] = (float)loss_l;
            my_loss += (double)loss_l;
        }
    }
    if (!DET) loss_finish(v, my_loss, n, loss_out);
}

// ---------------------------------------------------------------------------------------------
// matrix factorization
// ---------------------------------------------------------------------------------------------
// A warp keeps MF_DEPTH items in flight: the stored rows of the next MF_DEPTH items are already on their
// way (and the keys of the MF_DEPTH after those) while it does the dot product and the updates of the
// current one.  The workload is bound by DRAM: what counts is how many row fetches are outstanding.
#ifndef NUPS_MF_DEPTH
#define NUPS_MF_DEPTH 2
#endif
constexpr int MF_DEPTH = NUPS_MF_DEPTH;

template <bool HOT, bool DET, int CH, bool CLIP>
__global__ void __launch_bounds__(128, MF_DEPTH <= 2 ? 6 : (MF_DEPTH <= 4 ? 4 : 2))      // the grid is sized for this many blocks per SM
mf_kernel(View v, const uint32_t* __restrict__ rowk, const uint32_t* __restrict__ colk, const float* __restrict__ x,
          uint64_t n, float lr, float l2, float* __restrict__ upd, uint32_t* __restrict__ ukeys,
          float* __restrict__ loss_item, float* __restrict__ loss_out, float2* __restrict__ clip_item)
{
    grid_dependency_wait();
    const unsigned lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t nwarps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    const uint32_t L4 = v.L4;
    const float4* val4 = (const float4*)v.val;
    const float4* slab4 = (const float4*)v.dval;
    double my_loss = 0.0;
    const float bound = CLIP ? clip_bound(v) : 0.f;
    float my_clip = 0.f;
    unsigned my_clipped = 0;

    // ring A: keys and cell values of the items 2*MF_DEPTH .. MF_DEPTH+1 steps ahead
    // ring B: keys, slots and stored rows of the items MF_DEPTH .. 1 steps ahead
    uint32_t kiA[MF_DEPTH], kjA[MF_DEPTH], kiB[MF_DEPTH], kjB[MF_DEPTH];
    float xA[MF_DEPTH], xB[MF_DEPTH];
    int siB[MF_DEPTH], sjB[MF_DEPTH];
    float4 wB[MF_DEPTH][CH], hB[MF_DEPTH][CH];
    auto load_keys = [&](int u, uint64_t i) {
        if (i < n) { kiA[u] = rowk[i]; kjA[u] = colk[i]; xA[u] = x[i]; }
        else { kiA[u] = NUPS_INVALID_KEY; kjA[u] = NUPS_INVALID_KEY; xA[u] = 0.f; }
    };
    auto fetch_rows = [&](int u) {
        kiB[u] = kiA[u]; kjB[u] = kjA[u]; xB[u] = xA[u];
        const bool ok = kiB[u] < v.num_keys && kjB[u] < v.num_keys;
        siB[u] = (HOT && ok) ? __ldg(v.slot_of + kiB[u]) : -1;
        sjB[u] = (HOT && ok) ? __ldg(v.slot_of + kjB[u]) : -1;
#pragma unroll
        for (int m = 0; m < CH; ++m) {
            const uint32_t c = lane + 32 * m;
            wB[u][m] = make_float4(0.f, 0.f, 0.f, 0.f);
            hB[u][m] = wB[u][m];
            if (ok && c < L4) {
                wB[u][m] = val4[(uint64_t)kiB[u] * L4 + c];
                hB[u][m] = val4[(uint64_t)kjB[u] * L4 + c];
            }
        }
    };
#pragma unroll
    for (int u = 0; u < MF_DEPTH; ++u) load_keys(u, warp + (uint64_t)u * nwarps);
#pragma unroll
    for (int u = 0; u < MF_DEPTH; ++u) fetch_rows(u);
#pragma unroll
    for (int u = 0; u < MF_DEPTH; ++u) load_keys(u, warp + (uint64_t)(MF_DEPTH + u) * nwarps);

    for (uint64_t i0 = warp; i0 < n; i0 += (uint64_t)MF_DEPTH * nwarps) {
#pragma unroll
        for (int u = 0; u < MF_DEPTH; ++u) {
            const uint64_t i = i0 + (uint64_t)u * nwarps;
            if (i >= n) break;
            // take over what ring B fetched for this item, then refill both rings before computing
            const uint32_t ki = kiB[u], kj = kjB[u];
            const float xv = xB[u];
            const int si = siB[u], sj = sjB[u];
            float4 w[CH], h[CH];
#pragma unroll
            for (int m = 0; m < CH; ++m) { w[m] = wB[u][m]; h[m] = hB[u][m]; }
            fetch_rows(u);
            load_keys(u, i + 2ull * MF_DEPTH * nwarps);

            const uint32_t q = worker_of_item(i, n, v.R);
            const bool ok = ki < v.num_keys && kj < v.num_keys;
            if (DET && lane == 0) {
                ukeys[2 * i] = ok ? ki : NUPS_INVALID_KEY;
                ukeys[2 * i + 1] = ok ? kj : NUPS_INVALID_KEY;
            }
            if (!ok) {
                if (lane == 0) { flag_bad_key(v); if (DET) loss_item[i] = 0.f; if (DET && CLIP) clip_item[i] = make_float2(0.f, 0.f); }
                continue;
            }
            const uint64_t pw = si >= 0 ? ((uint64_t)q * v.Hcap + (unsigned)si) * L4 : 0;
            const uint64_t ph = sj >= 0 ? ((uint64_t)q * v.Hcap + (unsigned)sj) * L4 : 0;
            float dot = 0.f;
#pragma unroll
            for (int m = 0; m < CH; ++m) {
                const uint32_t c = lane + 32 * m;
                if (c < L4) {
                    if (HOT && si >= 0) w[m] = add4(w[m], slab4[pw + c]);       // the worker's pending replica updates
                    if (HOT && sj >= 0) h[m] = add4(h[m], slab4[ph + c]);
                }
                dot += w[m].x * h[m].x + w[m].y * h[m].y + w[m].z * h[m].z + w[m].w * h[m].w;
            }
            const float err = xv - warp_sum(dot);
            float fw = lr, fh = lr;                                 // learning rate times the clipping factor
            if (CLIP && (si >= 0 || sj >= 0)) {
                float nw2 = 0.f, nh2 = 0.f;
#pragma unroll
                for (int m = 0; m < CH; ++m) {
                    if (lane + 32 * m < L4) {
                        const float4 a = make_float4(err * h[m].x - l2 * w[m].x, err * h[m].y - l2 * w[m].y,
                                                     err * h[m].z - l2 * w[m].z, err * h[m].w - l2 * w[m].w);
                        const float4 b = make_float4(err * w[m].x - l2 * h[m].x, err * w[m].y - l2 * h[m].y,
                                                     err * w[m].z - l2 * h[m].z, err * w[m].w - l2 * h[m].w);
                        nw2 += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
                        nh2 += b.x * b.x + b.y * b.y + b.z * b.z + b.w * b.w;
                    }
                }
                float applied = 0.f, f;
                if (si >= 0) { applied += clip_norm(lr * sqrtf(warp_sum(nw2)), bound, &f); fw = lr * f; }
                if (sj >= 0) { applied += clip_norm(lr * sqrtf(warp_sum(nh2)), bound, &f); fh = lr * f; }
                const unsigned hot_roles = (si >= 0 ? 1u : 0u) + (sj >= 0 ? 1u : 0u);
                if (DET) { if (lane == 0) clip_item[i] = make_float2(applied, (float)hot_roles); }
                else { my_clip += applied; my_clipped += hot_roles; }
            } else if (CLIP && DET && lane == 0) {
                clip_item[i] = make_float2(0.f, 0.f);
            }
            float* ow = DET ? upd + (2 * i) * (uint64_t)L4 * 4 : (si >= 0 ? v.dval + pw * 4 : v.val + (uint64_t)ki * L4 * 4);
            float* oh = DET ? upd + (2 * i + 1) * (uint64_t)L4 * 4
                            : (sj >= 0 ? v.dval + ph * 4 : v.val + (uint64_t)kj * L4 * 4);
#pragma unroll
            for (int m = 0; m < CH; ++m) {
                const uint32_t c = lane + 32 * m;
                if (c < L4) {
                    const float4 dw = make_float4(fw * (err * h[m].x - l2 * w[m].x), fw * (err * h[m].y - l2 * w[m].y),
                                                  fw * (err * h[m].z - l2 * w[m].z), fw * (err * h[m].w - l2 * w[m].w));
                    const float4 dh = make_float4(fh * (err * w[m].x - l2 * h[m].x), fh * (err * w[m].y - l2 * h[m].y),
                                                  fh * (err * w[m].z - l2 * h[m].z), fh * (err * w[m].w - l2 * h[m].w));
                    if (DET) { ((float4*)ow)[c] = dw; ((float4*)oh)[c] = dh; }
                    else { red_add_v4(ow + 4 * c, dw); red_add_v4(oh + 4 * c, dh); }
                }
            }
            if (lane == 0) {
                if (!DET) {
                    if (si >= 0) mark_dirty(v, q, si);
                    if (sj >= 0) mark_dirty(v, q, sj);
                }
                if (v.count) {
                    note_access(v, ki, si, DET ? 1u : 2u);
                    note_access(v, kj, sj, DET ? 1u : 2u);
                }
                if (v.own) { mark_localize(v, ki, q); mark_localize(v, kj, q); }
                if (DET) loss_item[i] = err * err;
            }
            my_loss += (double)(err * err);
        }
    }
    if (!DET) loss_finish(v, my_loss, n, loss_out);
    if (CLIP && !DET) clip_finish(v, (double)my_clip, my_clipped);
}

// the finished step's clipping statistics join those of the earlier steps.  Deterministic mode: the
// per-item values (x = norms applied, y = how many) are summed in a fixed order first.
__global__ void clip_fold_kernel(DevStat* st, const float2* __restrict__ clip_item, uint64_t n)
{
    __shared__ double sh_s[256];
    __shared__ unsigned long long sh_c[256];
    double sm = 0.0;
    unsigned long long cn = 0;
    if (clip_item) {
        for (uint64_t i = threadIdx.x; i < n; i += 256) { sm += (double)clip_item[i].x; cn += (unsigned long long)clip_item[i].y; }
    }
    sh_s[threadIdx.x] = sm; sh_c[threadIdx.x] = cn;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) { sh_s[threadIdx.x] += sh_s[threadIdx.x + o]; sh_c[threadIdx.x] += sh_c[threadIdx.x + o]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        st->clip_sum += sh_s[0] + st->clip_step_sum;
        st->clip_cnt += sh_c[0] + st->clip_step_cnt;
        st->clip_step_sum = 0.0;
        st->clip_step_cnt = 0;
    }
}

// mean of the per-item losses, summed in a fixed order
__global__ void loss_mean_kernel(const float* __restrict__ loss_item, uint64_t n, float* __restrict__ out)
{
    __shared__ double sh[256];
    double s = 0.0;
    for (uint64_t i = threadIdx.x; i < n; i += 256) s += (double)loss_item[i];
    sh[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *out = (float)(sh[0] / (double)(n ? n : 1));
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
struct StepBuffers {
    float2* clip_item;      // deterministic mode with clipping: per item (norms applied, how many)
    float* loss_item;
    uint32_t* ukeys;
    float* uval;
    float* uacc;
    char* push_scratch;
};

static nups_status step_buffers(nups_store* s, uint64_t n, uint64_t per, bool two_tables, StepBuffers* b)
{
    const bool det = s->cfg.deterministic;
    uint64_t rows = n * per;
    size_t row_bytes = (size_t)rows * s->L * sizeof(float);
    const bool clip = det && s->cfg.clip_factor > 0.f && s->H;
    size_t need = align256(n * 4) + (clip ? align256(n * 8) : 0);
    if (det) need += align256(rows * 4) + align256(row_bytes) * (two_tables ? 2 : 1) + nups_push_scratch_bytes(s, rows);
    char* sc;
    nups_status rc = nups_scratch(s, need, &sc);
    if (rc != NUPS_OK) return rc;
    b->loss_item = (float*)sc; sc += align256(n * 4);
    b->clip_item = nullptr;
    if (clip) { b->clip_item = (float2*)sc; sc += align256(n * 8); }
    b->ukeys = nullptr; b->uval = nullptr; b->uacc = nullptr; b->push_scratch = nullptr;
    if (det) {
        b->ukeys = (uint32_t*)sc; sc += align256(rows * 4);
        b->uval = (float*)sc; sc += align256(row_bytes);
        if (two_tables) { b->uacc = (float*)sc; sc += align256(row_bytes); }
        b->push_scratch = sc;
    }
    return NUPS_OK;
}

static nups_status step_finish(nups_store* s, uint64_t n, uint64_t per, const StepBuffers& b,
                               float* d_loss_out, cudaStream_t st, bool loss_done_in_kernel = false, bool clips = false)
{
    nups_status rc;
    if (s->cfg.deterministic) {
        rc = nups_push_with_scratch(s, b.ukeys, n * per, (uint32_t)per, b.uval, b.uacc, b.push_scratch, st);
        if (rc != NUPS_OK) return rc;
    }
    if (d_loss_out && !loss_done_in_kernel) {
        loss_mean_kernel<<<1, 256, 0, st>>>(b.loss_item, n, d_loss_out);
        LAUNCH_CHECK(s);
    }
    if (clips && s->cfg.clip_factor > 0.f && s->H) {
        clip_fold_kernel<<<1, 256, 0, st>>>(s->st, b.clip_item, n);
        LAUNCH_CHECK(s);
    }
    s->steps++;
    if (s->cfg.sync_interval && s->steps % s->cfg.sync_interval == 0) return nups_sync_internal(s, st);
    return NUPS_OK;
}

// 4 warps per block, one item per warp per pass; at most `blocks_per_sm` blocks per SM, so that the grid is
// resident at once and a warp with several items can prefetch for its next one
static unsigned step_grid(const nups_store* s, uint64_t n, unsigned blocks_per_sm = 16)
{
    unsigned cap = (unsigned)s->sm_count * blocks_per_sm;
    if (cap > NUPS_MAX_STEP_BLOCKS) cap = NUPS_MAX_STEP_BLOCKS;
    return grid_for(n, 4, cap);
}

#define DISPATCH_CH(L4, ...)                                      \
    do {                                                          \
        if ((L4) <= 32) { constexpr int CH = 1; __VA_ARGS__; }    \
        else if ((L4) <= 64) { constexpr int CH = 2; __VA_ARGS__; } \
        else if ((L4) <= 96) { constexpr int CH = 3; __VA_ARGS__; } \
        else { constexpr int CH = 4; __VA_ARGS__; }               \
    } while (0)

#define DISPATCH_CLIP(s, ...)                                                                  \
    do {                                                                                     \
        if ((s)->cfg.clip_factor > 0.f && (s)->H) { constexpr bool CLIP = true; __VA_ARGS__; } \
        else { constexpr bool CLIP = false; __VA_ARGS__; }                                   \
    } while (0)

#define DISPATCH_MODE(s, ...)                                                                \
    do {                                                                                     \
        if ((s)->H) {                                                                        \
            if ((s)->cfg.deterministic) { constexpr bool HOT = true, DET = true; __VA_ARGS__; } \
            else { constexpr bool HOT = true, DET = false; __VA_ARGS__; }                    \
        } else {                                                                             \
            if ((s)->cfg.deterministic) { constexpr bool HOT = false, DET = true; __VA_ARGS__; } \
            else { constexpr bool HOT = false, DET = false; __VA_ARGS__; }                   \
        }                                                                                    \
    } while (0)

// resident blocks per multiprocessor of a kernel variant at a shared-memory size, asked of the runtime once and kept
template <class Query>
static cudaError_t resident_blocks(const void* fn, size_t smem, int* out, Query query)
{
    struct Entry { const void* fn; size_t smem; int fit; };
    static std::mutex mu;
    static std::vector<Entry> seen;
    std::lock_guard<std::mutex> g(mu);
    for (const Entry& e : seen)
        if (e.fn == fn && e.smem == smem) { *out = e.fit; return cudaSuccess; }
    cudaError_t rc = query(out);
    if (rc == cudaSuccess) seen.push_back({fn, smem, *out});
    return rc;
}

// launch of the fused skip-gram kernel over `group` consecutive steps of n pairs (group > 1: fast mode only;
// the negatives of all those steps lie back to back at s->last_negs, per-step losses go to loss_acc)
static nups_status sgns_launch(nups_store* s, const uint32_t* d_center, const uint32_t* d_context, uint64_t n, uint32_t K,
                               float lr, const StepBuffers& b, float* d_loss_out, uint32_t group,
                               unsigned long long* loss_acc, cudaStream_t st)
{
    View v = nups_view(s);
    const bool clip_on = s->cfg.clip_factor > 0.f && s->H;
    if (K == 3 && !s->cfg.deterministic && !s->cfg.count_accesses && !s->own && !clip_on) {
        // fast mode, nothing to count or move: the kernel that keeps rows in registers and sums runs of one centre word
        cudaError_t e = cudaSuccess;
        DISPATCH_CH(v.L4, {
            auto kern = s->H ? sgns_runs_kernel<true, CH> : sgns_runs_kernel<false, CH>;
            int fit = 0;
            e = resident_blocks((const void*)kern, 0, &fit, [&](int* out) {
                return cudaOccupancyMaxActiveBlocksPerMultiprocessor(out, kern, SGNS_RUN_THREADS, 0); });
            if (e == cudaSuccess) {
                if (fit < 1) fit = 1;
                const uint64_t items = n * group;
                const uint64_t blocks_needed = (items + SGNS_RUN_THREADS / 32 - 1) / (SGNS_RUN_THREADS / 32);
                const uint64_t cap = (uint64_t)s->sm_count * (unsigned)fit;
                const unsigned grid = (unsigned)(blocks_needed < cap ? blocks_needed : cap);
                nups_time_begin(s, st, NUPS_TIMED_STEP);
                nups_launch_dependent(kern, grid, SGNS_RUN_THREADS, 0, st, v, d_center, d_context, s->last_negs, n, lr, d_loss_out, group, loss_acc);
                nups_time_end(s, st);
            }
        });
        if (e != cudaSuccess) return nups_cuda_fail(e, "skip-gram kernel set-up");
        LAUNCH_CHECK(s);
        return NUPS_OK;
    }
    const uint32_t cols = ((v.L4 + 31) / 32) * 32, per = K + 2;    // a warp's staging area: per rows of cols chunks
    const size_t smem = (size_t)per * cols * sizeof(float4) * SGNS_WARPS;
    if (smem > (size_t)s->max_smem - 4096) return NUPS_EINVAL;
    // as many blocks as fit a multiprocessor's shared memory (each also holds about 2.5 KB besides its rows)
    unsigned per_sm = (unsigned)(((size_t)228 * 1024) / (smem + 2560));
    if (per_sm > 32) per_sm = 32;
    if (per_sm < 1) per_sm = 1;
    const uint64_t items = n * group;
    const uint64_t blocks_needed = (items + SGNS_WARPS - 1) / SGNS_WARPS;
    cudaError_t e = cudaSuccess;
#define NUPS_SGNS_GO(KT_)                                                                                              \
    DISPATCH_CH(v.L4, DISPATCH_MODE(s, DISPATCH_CLIP(s, {                                                              \
        auto kern = sgns_kernel<HOT, DET, KT_, CH, (HOT && CLIP)>;                                                     \
        if (smem > 48 * 1024)                                                                                          \
            e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, s->max_smem - 4096);           \
        int fit = 0;       /* registers may allow fewer resident blocks than shared memory does: no second wave */ \
        if (e == cudaSuccess) e = resident_blocks((const void*)kern, smem, &fit, [&](int* out) {                       \
            return cudaOccupancyMaxActiveBlocksPerMultiprocessor(out, kern, 32 * SGNS_WARPS, smem); });                \
        if (e == cudaSuccess) {                                                                                        \
            if (fit >= 1 && (unsigned)fit < per_sm) per_sm = (unsigned)fit;                                            \
            const uint64_t cap = (uint64_t)s->sm_count * per_sm;                                                       \
            const unsigned grid = (unsigned)(blocks_needed < cap ? blocks_needed : cap);                               \
            nups_time_begin(s, st, NUPS_TIMED_STEP);                                                                                    \
            nups_launch_dependent(kern, grid, 32 * SGNS_WARPS, smem, st, v, d_center, d_context, s->last_negs, n, K, lr, b.uval, b.ukeys, \
                                                      b.loss_item, d_loss_out, group,                                  \
                                                      loss_acc, b.clip_item);                                          \
            nups_time_end(s, st);                                                                                      \
        }                                                                                                              \
    })))
    if (K == 3) NUPS_SGNS_GO(3);
    else NUPS_SGNS_GO(0);
#undef NUPS_SGNS_GO
    if (e != cudaSuccess) return nups_cuda_fail(e, "skip-gram kernel set-up");
    LAUNCH_CHECK(s);
    return NUPS_OK;
}

static nups_status sgns_check(nups_store* s, const uint32_t* d_center, const uint32_t* d_context, uint64_t n, uint32_t K)
{
    if (!s || !d_center || !d_context || n == 0 || n * (uint64_t)(K + 2) >= (1ull << 32)) return NUPS_EINVAL;
    if (K > 30) return NUPS_EINVAL;                         // one lane per key of an item
    if (s->vb != 4) return NUPS_ESTATE;                     // the skip-gram step is single precision only
    if (s->L / 4 > SGNS_MAX_CHUNKS) return NUPS_EINVAL;     // four float4 chunks of a row per lane: at most 512 floats
    return NUPS_OK;
}

extern "C" nups_status nups_step_sgns(nups_store* s, const uint32_t* d_center, const uint32_t* d_context, uint64_t n,
                                      int32_t dist, uint32_t K, float lr, float* d_loss_out, void* stream)
{
    nups_status rc = sgns_check(s, d_center, d_context, n, K);
    if (rc != NUPS_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    rc = nups_draw_negatives(s, dist, n * K, st);
    if (rc != NUPS_OK) return rc;
    rc = nups_new_epoch(s, st);
    if (rc != NUPS_OK) return rc;
    StepBuffers b;
    rc = step_buffers(s, n, K + 2, false, &b);
    if (rc != NUPS_OK) return rc;
    rc = sgns_launch(s, d_center, d_context, n, K, lr, b, d_loss_out, 1, nullptr, st);
    if (rc != NUPS_OK) return rc;
    return step_finish(s, n, K + 2, b, d_loss_out, st, !s->cfg.deterministic, true);
}

// per-step losses of a grouped launch: fixed-point sums -> means, and the sums are cleared for the next group
__global__ void loss_group_kernel(unsigned long long* acc, uint32_t group, uint64_t n, float* loss_out)
{
    grid_dependency_wait();
    const uint32_t g = threadIdx.x;
    if (g >= group) return;
    unsigned long long sum = 0;
    for (uint32_t k = 0; k < LOSS_SLOTS; ++k) { sum += acc[k * LOSS_STEPS + g]; acc[k * LOSS_STEPS + g] = 0ull; }
    if (loss_out) loss_out[g] = (float)((double)sum / 65536.0 / (double)n);
}

extern "C" nups_status nups_run_sgns(nups_store* s, const uint32_t* d_center, const uint32_t* d_context, uint64_t n_total,
                                     uint64_t batch, int32_t dist, uint32_t K, float lr, float* d_loss_out, void* stream)
{
    if (batch == 0 || n_total == 0 || n_total % batch) return NUPS_EINVAL;
    nups_status rc = sgns_check(s, d_center, d_context, batch, K);
    if (rc != NUPS_OK) return rc;
    const uint64_t steps = n_total / batch;
    // where a step has side effects that must happen in step order (ordered pushes, access counts,
    // ownership changes), the steps are simply taken one by one
    if (s->cfg.deterministic || s->cfg.count_accesses || s->own) {
        for (uint64_t t = 0; t < steps; ++t) {
            rc = nups_step_sgns(s, d_center + t * batch, d_context + t * batch, batch, dist, K, lr,
                                d_loss_out ? d_loss_out + t : nullptr, stream);
            if (rc != NUPS_OK) return rc;
        }
        return NUPS_OK;
    }
    cudaStream_t st = (cudaStream_t)stream;
    unsigned long long* acc = (unsigned long long*)s->loss_partial;      // zero between launches
    StepBuffers b;
    b.loss_item = nullptr; b.clip_item = nullptr; b.ukeys = nullptr; b.uval = nullptr; b.uacc = nullptr;
    b.push_scratch = nullptr;
    // A replica merge that falls due while more steps of this call follow runs on a stream of its own, beside the
    // draw of the next steps' negatives (the draw touches neither replicas nor rows); the next step kernel waits for it.
    if (!s->side) {
        CK(cudaStreamCreateWithFlags(&s->side, cudaStreamNonBlocking));
        CK(cudaEventCreateWithFlags(&s->side_fork, cudaEventDisableTiming));
        CK(cudaEventCreateWithFlags(&s->side_join, cudaEventDisableTiming));
    }
    bool merge_in_flight = false;
    uint64_t t = 0;
    while (t < steps) {
        // one launch covers the steps up to the next replica merge, as far as their negatives are drawn already
        rc = nups_draw_negatives(s, dist, batch * K, st);                 // this step's negatives (may draw ahead)
        if (rc != NUPS_OK) return rc;
        if (merge_in_flight) {
            CK(cudaStreamWaitEvent(st, s->side_join, 0));
            merge_in_flight = false;
        }
        uint64_t group = 1;
        if (s->ahead_dist == dist && s->ahead_N == batch * K) group += s->ahead_total - s->ahead_next;
        if (group > steps - t) group = steps - t;
        if (s->cfg.sync_interval) {
            const uint64_t to_sync = s->cfg.sync_interval - s->steps % s->cfg.sync_interval;
            if (group > to_sync) group = to_sync;
        }
        if (group > LOSS_STEPS) group = LOSS_STEPS;
        if (group > 1) s->ahead_next += (uint32_t)(group - 1);            // those batches are handed out now
        rc = sgns_launch(s, d_center + t * batch, d_context + t * batch, batch, K, lr, b, nullptr, (uint32_t)group, acc, st);
        if (rc != NUPS_OK) return rc;
        nups_launch_dependent(loss_group_kernel, 1, LOSS_STEPS, 0, st, acc, (uint32_t)group, batch, d_loss_out ? d_loss_out + t : nullptr);
        LAUNCH_CHECK(s);
        if (s->cfg.clip_factor > 0.f && s->H) {
            clip_fold_kernel<<<1, 256, 0, st>>>(s->st, nullptr, 0);      // the launch's clipping statistics join the rest
            LAUNCH_CHECK(s);
        }
        s->steps += group;
        t += group;
        if (s->cfg.sync_interval && s->steps % s->cfg.sync_interval == 0) {
            if (t < steps) {
                CK(cudaEventRecord(s->side_fork, st));
                CK(cudaStreamWaitEvent(s->side, s->side_fork, 0));
                rc = nups_sync_internal(s, s->side);
                if (rc != NUPS_OK) return rc;
                CK(cudaEventRecord(s->side_join, s->side));
                merge_in_flight = true;
            } else {
                rc = nups_sync_internal(s, st);
                if (rc != NUPS_OK) return rc;
            }
        }
    }
    return NUPS_OK;
}

extern "C" nups_status nups_step_complex(nups_store* s, const uint32_t* d_h, const uint32_t* d_r, const uint32_t* d_t,
                                         uint64_t n, int32_t dist, uint32_t K, float lr, float eps, float* d_loss_out,
                                         void* stream)
{
    if (!s || !d_h || !d_r || !d_t || n == 0 || n * (uint64_t)(K + 3) >= (1ull << 32)) return NUPS_EINVAL;
    if (!s->acc || s->value_len / 4 > CPX_THREADS || (s->value_len & 3) || K > 30) return NUPS_EINVAL;    // one thread per component pair, one lane per score
    cudaStream_t st = (cudaStream_t)stream;
    nups_status rc = nups_draw_negatives(s, dist, n * K, st);
    if (rc != NUPS_OK) return rc;
    rc = nups_new_epoch(s, st);
    if (rc != NUPS_OK) return rc;
    StepBuffers b;
    rc = step_buffers(s, n, K + 3, true, &b);
    if (rc != NUPS_OK) return rc;
    View v = nups_view(s);
    // shared memory: the value and the accumulator row of every role
    const size_t smem = (size_t)2 * (K + 3) * s->L * sizeof(float);
    if (smem > (size_t)s->max_smem - 4096) return NUPS_EINVAL;
    unsigned per_sm = (unsigned)(((size_t)s->max_smem - 1024) / (smem + 2048));
    if (per_sm > 4) per_sm = 4;
    if (per_sm < 1) per_sm = 1;
    uint64_t want = n < (uint64_t)s->sm_count * per_sm ? n : (uint64_t)s->sm_count * per_sm;
    unsigned grid = (unsigned)want;
    const int hi = s->H ? 1 : 0, di = s->cfg.deterministic ? 1 : 0, ri = K + 1 <= (uint32_t)CPX_NS ? 1 : 0, fi = s->vb == 8 ? 1 : 0;
    if (fi && grid > (unsigned)s->sm_count * 2) grid = (unsigned)s->sm_count * 2;      // the 8-byte variant: two blocks per multiprocessor
    cudaError_t e = cudaSuccess;
    nups_time_begin(s, st, NUPS_TIMED_STEP);
#define NUPS_CPX_GO(RED16_, F64_)                                                                                    \
    DISPATCH_MODE(s, {                                                                                               \
        auto kern = complex_kernel<HOT, DET, RED16_, F64_>;                                                          \
        if (!s->complex_smem_opted[hi][di][ri][fi]) {                                                                \
            e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, s->max_smem - 4096);         \
            s->complex_smem_opted[hi][di][ri][fi] = (e == cudaSuccess);                                              \
        }                                                                                                            \
        if (e == cudaSuccess)                                                                                        \
            nups_launch_dependent(kern, grid, CPX_THREADS, smem, st, v, d_h, d_r, d_t, s->last_negs, n, K, lr, eps, b.uval, b.uacc, \
                                                  b.ukeys, b.loss_item, d_loss_out);                                 \
    })
    if (fi) { if (ri) NUPS_CPX_GO(true, true); else NUPS_CPX_GO(false, true); }
    else { if (ri) NUPS_CPX_GO(true, false); else NUPS_CPX_GO(false, false); }
#undef NUPS_CPX_GO
    nups_time_end(s, st);
    if (e != cudaSuccess) return nups_cuda_fail(e, "cudaFuncSetAttribute");
    LAUNCH_CHECK(s);
    return step_finish(s, n, K + 3, b, d_loss_out, st, !s->cfg.deterministic);
}

// ---------------------------------------------------------------------------------------------
// matrix factorization over cells that come column by column (Section 5.1: every worker visits its cells
// by column, to create locality in the accesses to column parameters).  Fast mode only.
// A warp works on a stretch of consecutive cells.  The keys, cell values and replica slots of 32 cells are
// loaded by the 32 lanes at once, one window ahead.  The rows of the row keys are fetched MF_RUN_DEPTH cells
// ahead into a register ring.  The row of the column key stays in registers while the column stays the same
// (the next column's row is fetched one cell before it is needed), and the column's update is summed in
// registers and added once when the column changes: a column's row costs one read and one reduction per
// stretch instead of one per cell.  Within a stretch the cells of a column all see the column's row from
// before the stretch (the batch semantics of the deterministic mode); rows of row keys are read as they are.
// ---------------------------------------------------------------------------------------------
constexpr int MF_RUN_DEPTH = 4;           // divides 32
constexpr int MF_RUN_BLOCKS = 5;          // resident blocks per multiprocessor the grid is sized for

template <bool HOT, int CH, bool CLIP>
__global__ void __launch_bounds__(128, MF_RUN_BLOCKS)
mf_runs_kernel(View v, const uint32_t* __restrict__ rowk, const uint32_t* __restrict__ colk, const float* __restrict__ x,
               uint64_t n, float lr, float l2, float* __restrict__ loss_out)
{
    grid_dependency_wait();
    constexpr unsigned FULL = 0xFFFFFFFFu;
    const unsigned lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t nwarps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    const uint32_t L4 = v.L4;
    const float4* val4 = (const float4*)v.val;
    const float4* slab4 = (const float4*)v.dval;
    double my_loss = 0.0;
    const float bound = CLIP ? clip_bound(v) : 0.f;
    float my_clip = 0.f;
    unsigned my_clipped = 0;
    const uint64_t stretch = (n + nwarps - 1) / nwarps;
    const uint64_t first = warp * stretch < n ? warp * stretch : n;
    const uint64_t last = first + stretch < n ? first + stretch : n;            // this warp's cells: [first, last)

    // one window = 32 consecutive cells, lane l holds cell l: keys (row key invalid when either key is),
    // cell value, replica slots
    struct Window { uint32_t ki, kj; float x; int si, sj; };
    auto load_window = [&](uint64_t base) {
        Window w = {NUPS_INVALID_KEY, NUPS_INVALID_KEY, 0.f, -1, -1};
        const uint64_t i = base + lane;
        if (i < last) {
            const uint32_t ki = rowk[i], kj = colk[i];
            w.x = x[i];
            if (ki < v.num_keys && kj < v.num_keys) {
                w.ki = ki; w.kj = kj;
                if (HOT) { w.si = __ldg(v.slot_of + ki); w.sj = __ldg(v.slot_of + kj); }
            } else {
                flag_bad_key(v);
            }
        }
        return w;
    };
    Window cur = load_window(first), nxt = load_window(first + 32);
    // cell t of the current window (t < 32) or of the next one (32 <= t < 64)
    auto row_key_at = [&](uint32_t t) {
        const uint32_t a = __shfl_sync(FULL, cur.ki, t & 31), b = __shfl_sync(FULL, nxt.ki, t & 31);
        return t < 32 ? a : b;
    };
    auto col_key_at = [&](uint32_t t) {
        const uint32_t a = __shfl_sync(FULL, cur.kj, t & 31), b = __shfl_sync(FULL, nxt.kj, t & 31);
        return t < 32 ? a : b;
    };
    auto fetch_row = [&](float4 (&dst)[CH], uint32_t key) {
#pragma unroll
        for (int m = 0; m < CH; ++m) {
            const uint32_t c = lane + 32 * m;
            dst[m] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (key != NUPS_INVALID_KEY && c < L4) dst[m] = val4[(uint64_t)key * L4 + c];
        }
    };

    float4 ring[MF_RUN_DEPTH][CH];                       // stored rows of the row keys of the next cells
#pragma unroll
    for (int u = 0; u < MF_RUN_DEPTH; ++u) fetch_row(ring[u], row_key_at(u));
    uint32_t h_key = NUPS_INVALID_KEY, h_next_key = NUPS_INVALID_KEY;
    float4 h[CH], h_next[CH];                            // stored row of the current column, and of the one after it
    {
        const uint32_t k0 = col_key_at(0);
        fetch_row(h_next, k0);
        h_next_key = k0;
    }
    float* held_row = nullptr;                           // column row whose summed update is still in registers
    float4 held[CH];
    auto flush_held = [&]() {
        if (!held_row) return;
#pragma unroll
        for (int m = 0; m < CH; ++m) {
            const uint32_t c = lane + 32 * m;
            if (c < L4) red_add_v4(held_row + 4 * c, held[m]);
        }
        held_row = nullptr;
    };

    uint32_t q = worker_of_item(first < n ? first : 0, n, v.R);    // worker of the cell at hand, kept up as i grows
    uint64_t q_end = worker_first_item(q + 1, n, v.R);
    float window_loss = 0.f;
    for (uint64_t base = first; base < last; base += 32) {
        for (uint32_t t0 = 0; t0 < 32; t0 += MF_RUN_DEPTH) {
            if (base + t0 >= last) break;
#pragma unroll
            for (int u = 0; u < MF_RUN_DEPTH; ++u) {
                const uint32_t t = t0 + u;
                const uint64_t i = base + t;
                if (i >= last) break;
                const uint32_t ki = __shfl_sync(FULL, cur.ki, t), kj = __shfl_sync(FULL, cur.kj, t);
                const float xv = __shfl_sync(FULL, cur.x, t);
                const int si = __shfl_sync(FULL, cur.si, t), sj = __shfl_sync(FULL, cur.sj, t);
                float4 w[CH];
#pragma unroll
                for (int m = 0; m < CH; ++m) w[m] = ring[u][m];
                fetch_row(ring[u], row_key_at(t + MF_RUN_DEPTH));
                if (ki == NUPS_INVALID_KEY) continue;               // a bad key: flagged when the window was loaded
                if (kj != h_key) {
                    if (h_next_key != kj) { fetch_row(h_next, kj); h_next_key = kj; }
#pragma unroll
                    for (int m = 0; m < CH; ++m) h[m] = h_next[m];
                    h_key = kj;
                }
                {
                    const uint32_t kj1 = col_key_at(t + 1);
                    if (kj1 != NUPS_INVALID_KEY && kj1 != h_key && kj1 != h_next_key) { fetch_row(h_next, kj1); h_next_key = kj1; }
                }
                while (i >= q_end) q_end = worker_first_item(++q + 1, n, v.R);
                const uint64_t pw = si >= 0 ? ((uint64_t)q * v.Hcap + (unsigned)si) * L4 : 0;
                const uint64_t ph = sj >= 0 ? ((uint64_t)q * v.Hcap + (unsigned)sj) * L4 : 0;
                float4 hv[CH];
                float dot = 0.f;
#pragma unroll
                for (int m = 0; m < CH; ++m) {
                    const uint32_t c = lane + 32 * m;
                    hv[m] = h[m];
                    if (c < L4) {
                        if (HOT && si >= 0) w[m] = add4(w[m], slab4[pw + c]);       // the worker's pending replica updates
                        if (HOT && sj >= 0) hv[m] = add4(hv[m], slab4[ph + c]);
                    }
                    dot += w[m].x * hv[m].x + w[m].y * hv[m].y + w[m].z * hv[m].z + w[m].w * hv[m].w;
                }
                const float err = xv - warp_sum(dot);
                float fw = lr, fh = lr;                                 // learning rate times the clipping factor
                if (CLIP && (si >= 0 || sj >= 0)) {
                    float nw2 = 0.f, nh2 = 0.f;
#pragma unroll
                    for (int m = 0; m < CH; ++m) {
                        if (lane + 32 * m < L4) {
                            const float4 a = make_float4(err * hv[m].x - l2 * w[m].x, err * hv[m].y - l2 * w[m].y,
                                                         err * hv[m].z - l2 * w[m].z, err * hv[m].w - l2 * w[m].w);
                            const float4 b = make_float4(err * w[m].x - l2 * hv[m].x, err * w[m].y - l2 * hv[m].y,
                                                         err * w[m].z - l2 * hv[m].z, err * w[m].w - l2 * hv[m].w);
                            nw2 += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
                            nh2 += b.x * b.x + b.y * b.y + b.z * b.z + b.w * b.w;
                        }
                    }
                    float applied = 0.f, f;
                    if (si >= 0) { applied += clip_norm(lr * sqrtf(warp_sum(nw2)), bound, &f); fw = lr * f; }
                    if (sj >= 0) { applied += clip_norm(lr * sqrtf(warp_sum(nh2)), bound, &f); fh = lr * f; }
                    my_clip += applied;
                    my_clipped += (si >= 0 ? 1u : 0u) + (sj >= 0 ? 1u : 0u);
                }
                float* ow = si >= 0 ? v.dval + pw * 4 : v.val + (uint64_t)ki * L4 * 4;
                float* oh = sj >= 0 ? v.dval + ph * 4 : v.val + (uint64_t)kj * L4 * 4;
                if (held_row != oh) flush_held();
#pragma unroll
                for (int m = 0; m < CH; ++m) {
                    const uint32_t c = lane + 32 * m;
                    if (c < L4) {
                        const float4 dw = make_float4(fw * (err * hv[m].x - l2 * w[m].x), fw * (err * hv[m].y - l2 * w[m].y),
                                                      fw * (err * hv[m].z - l2 * w[m].z), fw * (err * hv[m].w - l2 * w[m].w));
                        const float4 dh = make_float4(fh * (err * w[m].x - l2 * hv[m].x), fh * (err * w[m].y - l2 * hv[m].y),
                                                      fh * (err * w[m].z - l2 * hv[m].z), fh * (err * w[m].w - l2 * hv[m].w));
                        red_add_v4(ow + 4 * c, dw);
                        held[m] = oh == held_row ? add4(held[m], dh) : dh;
                    }
                }
                held_row = oh;
                if (lane == 0) {
                    if (si >= 0) mark_dirty(v, q, si);
                    if (sj >= 0) mark_dirty(v, q, sj);
                    if (v.count) { note_access(v, ki, si, 2u); note_access(v, kj, sj, 2u); }
                    if (v.own) { mark_localize(v, ki, q); mark_localize(v, kj, q); }
                }
                window_loss += err * err;
            }
        }
        my_loss += (double)window_loss;
        window_loss = 0.f;
        cur = nxt;
        nxt = load_window(base + 64);
    }
    flush_held();
    loss_finish(v, my_loss, n, loss_out);
    if (CLIP) clip_finish(v, (double)my_clip, my_clipped);
}

// ---------------------------------------------------------------------------------------------
// matrix factorization on 8-byte values: one warp per cell, lanes stride over the row's values, everything
// in double precision.  (Plain: the single-precision kernels above are the tuned ones.)
// ---------------------------------------------------------------------------------------------
namespace {
template <bool HOT, bool DET>
__global__ void __launch_bounds__(128)
mf_f64_kernel(View v, const uint32_t* __restrict__ rowk, const uint32_t* __restrict__ colk, const float* __restrict__ x,
              uint64_t n, float lr, float l2, float* __restrict__ upd, uint32_t* __restrict__ ukeys,
              float* __restrict__ loss_item, float* __restrict__ loss_out)
{
    grid_dependency_wait();
    const unsigned lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t nwarps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    const uint32_t L = v.L4 * 2;                               // values per row
    const double* val = reinterpret_cast<const double*>(v.val);
    const double* slab = reinterpret_cast<const double*>(v.dval);
    double* uout = reinterpret_cast<double*>(upd);
    const double lrd = (double)lr, l2d = (double)l2;
    double my_loss = 0.0;
    for (uint64_t i = warp; i < n; i += nwarps) {
        const uint32_t ki = rowk[i], kj = colk[i];
        const bool ok = ki < v.num_keys && kj < v.num_keys;
        if (DET && lane == 0) {
            ukeys[2 * i] = ok ? ki : NUPS_INVALID_KEY;
            ukeys[2 * i + 1] = ok ? kj : NUPS_INVALID_KEY;
        }
        if (!ok) {
            if (lane == 0) { flag_bad_key(v); if (DET) loss_item[i] = 0.f; }
            continue;
        }
        const uint32_t q = worker_of_item(i, n, v.R);
        const int si = HOT ? __ldg(v.slot_of + ki) : -1, sj = HOT ? __ldg(v.slot_of + kj) : -1;
        const double* wrow = val + (uint64_t)ki * L;
        const double* hrow = val + (uint64_t)kj * L;
        const double* wpend = si >= 0 ? slab + ((uint64_t)q * v.Hcap + (unsigned)si) * L : nullptr;
        const double* hpend = sj >= 0 ? slab + ((uint64_t)q * v.Hcap + (unsigned)sj) * L : nullptr;
        double dot = 0.0;
        for (uint32_t e = lane; e < L; e += 32) {
            const double w = wrow[e] + (wpend ? wpend[e] : 0.0), h = hrow[e] + (hpend ? hpend[e] : 0.0);
            dot += w * h;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xFFFFFFFFu, dot, o);
        const double err = (double)x[i] - dot;
        double* ow = DET ? uout + (2 * i) * (uint64_t)L : reinterpret_cast<double*>(si >= 0 ? v.dval : v.val) +
                                                              (si >= 0 ? ((uint64_t)q * v.Hcap + (unsigned)si) * L : (uint64_t)ki * L);
        double* oh = DET ? uout + (2 * i + 1) * (uint64_t)L : reinterpret_cast<double*>(sj >= 0 ? v.dval : v.val) +
                                                                  (sj >= 0 ? ((uint64_t)q * v.Hcap + (unsigned)sj) * L : (uint64_t)kj * L);
        for (uint32_t e = lane; e < L; e += 32) {
            const double w = wrow[e] + (wpend ? wpend[e] : 0.0), h = hrow[e] + (hpend ? hpend[e] : 0.0);
            const double dw = lrd * (err * h - l2d * w), dh = lrd * (err * w - l2d * h);
            if (DET) { ow[e] = dw; oh[e] = dh; }
            else { atomicAdd(ow + e, dw); atomicAdd(oh + e, dh); }
        }
        if (lane == 0) {
            if (!DET) {
                if (si >= 0) mark_dirty(v, q, si);
                if (sj >= 0) mark_dirty(v, q, sj);
            }
            if (v.count) {
                note_access(v, ki, si, DET ? 1u : 2u);
                note_access(v, kj, sj, DET ? 1u : 2u);
            }
            if (v.own) { mark_localize(v, ki, q); mark_localize(v, kj, q); }
            if (DET) loss_item[i] = (float)(err * err);
        }
        my_loss += err * err;
    }
    if (!DET) loss_finish(v, my_loss, n, loss_out);
}
}  // namespace

static nups_status mf_step(nups_store* s, const uint32_t* d_row, const uint32_t* d_col, const float* d_x,
                           uint64_t n, float lr, float l2, float* d_loss_out, void* stream, bool cells_by_column)
{
    if (!s || !d_row || !d_col || !d_x || n == 0 || n * 2 >= (1ull << 32)) return NUPS_EINVAL;
    if (s->vb == 4 && s->L / 4 > 128) return NUPS_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    s->last_negs_n = 0;
    nups_status rc = nups_new_epoch(s, st);
    if (rc != NUPS_OK) return rc;
    StepBuffers b;
    rc = step_buffers(s, n, 2, false, &b);
    if (rc != NUPS_OK) return rc;
    View v = nups_view(s);
    const bool by_column = cells_by_column && !s->cfg.deterministic;    // the ordered mode is the same for any order
    nups_time_begin(s, st, NUPS_TIMED_STEP);
    if (s->vb == 8) {
        const unsigned grid = step_grid(s, n, 8);
        DISPATCH_MODE(s, nups_launch_dependent(mf_f64_kernel<HOT, DET>, grid, 128, 0, st, v, d_row, d_col, d_x, n, lr, l2, b.uval, b.ukeys,
                                                                      b.loss_item, d_loss_out));
    } else if (by_column) {
        const unsigned grid = step_grid(s, n, MF_RUN_BLOCKS);
        DISPATCH_CLIP(s, DISPATCH_CH(v.L4, {
            if (s->H) nups_launch_dependent(mf_runs_kernel<true, CH, CLIP>, grid, 128, 0, st, v, d_row, d_col, d_x, n, lr, l2, d_loss_out);
            else nups_launch_dependent(mf_runs_kernel<false, CH, false>, grid, 128, 0, st, v, d_row, d_col, d_x, n, lr, l2, d_loss_out);
        }));
    } else {
        const unsigned grid = step_grid(s, n, MF_DEPTH <= 2 ? 6 : (MF_DEPTH <= 4 ? 4 : 2));   // resident blocks at that depth's register use
        DISPATCH_MODE(s, DISPATCH_CLIP(s, DISPATCH_CH(v.L4, nups_launch_dependent(mf_kernel<HOT, DET, CH, (HOT && CLIP)>, grid, 128, 0, st,
            v, d_row, d_col, d_x, n, lr, l2, b.uval, b.ukeys, b.loss_item, d_loss_out, b.clip_item))));
    }
    nups_time_end(s, st);
    LAUNCH_CHECK(s);
    return step_finish(s, n, 2, b, d_loss_out, st, !s->cfg.deterministic, true);
}

extern "C" nups_status nups_step_mf(nups_store* s, const uint32_t* d_row, const uint32_t* d_col, const float* d_x,
                                    uint64_t n, float lr, float l2, float* d_loss_out, void* stream)
{
    return mf_step(s, d_row, d_col, d_x, n, lr, l2, d_loss_out, stream, false);
}

extern "C" nups_status nups_step_mf_by_column(nups_store* s, const uint32_t* d_row, const uint32_t* d_col,
                                              const float* d_x, uint64_t n, float lr, float l2, float* d_loss_out,
                                              void* stream)
{
    return mf_step(s, d_row, d_col, d_x, n, lr, l2, d_loss_out, stream, true);
}

extern "C" nups_status nups_get_clip_stats(nups_store* s, double* h_sum, uint64_t* h_count, void* stream)
{
    if (!s || !h_sum || !h_count) return NUPS_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    DevStat d;
    CK(cudaMemcpyAsync(&d, s->st, sizeof(DevStat), cudaMemcpyDeviceToHost, st));
    CK(cudaStreamSynchronize(st));
    *h_sum = d.clip_sum;
    *h_count = d.clip_cnt;
    return NUPS_OK;
}
