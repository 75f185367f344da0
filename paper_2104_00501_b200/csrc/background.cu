// Time-based replica synchronisation (NuPS Section 3.2: replicas are synchronised periodically by a
// background thread, staleness bounded by time rather than by a logical clock; Section 5.6 varies the
// period).  A host thread owned by the store enqueues a merge of all replicas every `period` on a
// stream of its own, so the merge overlaps whatever the caller's streams are running and never
// blocks a worker.
//
// The merge must tolerate updates that land while it runs.  It therefore never stores to a replica:
// for every replicated row and worker it reads the pending update x, takes exactly x back out of the
// replica with a reduction (an update added in the meantime stays), and adds the sum over the workers
// to the stored row with a reduction.  No update is lost or applied twice; a reader may for a moment
// see the stored row without an x that has already left its replica (a stale read, which bounded
// staleness allows).  It sweeps every replicated slot instead of trusting the touched flags (setting a
// flag and adding to the replica are not one atomic step), and skips rows that are all zero, so only
// updated parameters cost more than the read.
#include <chrono>
#include <condition_variable>
#include <mutex>
#include <new>
#include <thread>

#include "nups_internal.cuh"

struct nups_background {
    std::thread th;
    std::mutex mu;                 // held while a merge is enqueued and while the hot set is rebuilt
    std::condition_variable cv;
    bool stop = false;
    uint32_t period_us = 0;
    cudaStream_t stream = nullptr;
    cudaEvent_t merged = nullptr;  // end of the most recent background merge
    cudaEvent_t fence = nullptr;   // end of caller-stream work that background merges must not overtake
    bool any_merge = false;
    uint64_t merges = 0;
};

__global__ void __launch_bounds__(256)
merge_async_kernel(float* __restrict__ val, float* __restrict__ acc, float* dval, float* dacc,
                   const uint32_t* __restrict__ hot_keys, uint64_t H, uint64_t Hcap, uint32_t R, uint32_t L4)
{
    const uint64_t e = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= H * L4) return;
    const uint64_t slot = e / L4;
    const uint32_t c = (uint32_t)(e % L4);
    const uint32_t key = hot_keys[slot];
    for (int which = 0; which < 2; ++which) {
        float* table = which ? acc : val;
        float* slab = which ? dacc : dval;
        if (!table || !slab) continue;
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
        bool any = false;
        for (uint32_t r = 0; r < R; ++r) {
            float* p = slab + (((uint64_t)r * Hcap + slot) * L4 + c) * 4;
            const float4 x = __ldcg(reinterpret_cast<const float4*>(p));
            if (x.x != 0.f || x.y != 0.f || x.z != 0.f || x.w != 0.f) {
                red_add_v4(p, make_float4(-x.x, -x.y, -x.z, -x.w));
                sum = add4(sum, x);
                any = true;
            }
        }
        if (any) red_add_v4(table + ((uint64_t)key * L4 + c) * 4, sum);
    }
}

static void background_loop(nups_store* s)
{
    nups_background* bg = s->bg;
    cudaSetDevice(s->device);
    std::unique_lock<std::mutex> lk(bg->mu);
    while (!bg->stop) {
        if (bg->period_us == 0) {
            bg->cv.wait(lk);
            continue;
        }
        bg->cv.wait_for(lk, std::chrono::microseconds(bg->period_us));
        if (bg->stop || bg->period_us == 0 || s->H == 0) continue;
        // one merge at a time: if the previous one has not finished, this tick is skipped
        if (bg->any_merge && cudaEventQuery(bg->merged) != cudaSuccess) { cudaGetLastError(); continue; }
        const uint64_t work = s->H * (s->L / 4);
        merge_async_kernel<<<grid_for(work, 256), 256, 0, bg->stream>>>(s->val, s->acc, s->dval, s->dacc, s->hot_keys, s->H,
                                                                       s->Hcap, s->R, s->L / 4);
        if (cudaGetLastError() == cudaSuccess && cudaEventRecord(bg->merged, bg->stream) == cudaSuccess) {
            bg->any_merge = true;
            bg->merges++;
        }
    }
}

nups_status nups_background_start(nups_store* s, uint32_t period_us)
{
    nups_background* bg = new (std::nothrow) nups_background();
    if (!bg) return NUPS_ENOMEM;
    if (cudaStreamCreateWithFlags(&bg->stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&bg->merged, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&bg->fence, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        if (bg->stream) cudaStreamDestroy(bg->stream);
        if (bg->merged) cudaEventDestroy(bg->merged);
        delete bg;
        return NUPS_ECUDA;
    }
    bg->period_us = period_us;
    s->bg = bg;
    bg->th = std::thread(background_loop, s);
    return NUPS_OK;
}

void nups_background_stop(nups_store* s)
{
    nups_background* bg = s->bg;
    if (!bg) return;
    {
        std::lock_guard<std::mutex> g(bg->mu);
        bg->stop = true;
    }
    bg->cv.notify_all();
    bg->th.join();
    cudaStreamSynchronize(bg->stream);
    cudaStreamDestroy(bg->stream);
    cudaEventDestroy(bg->merged);
    cudaEventDestroy(bg->fence);
    delete bg;
    s->bg = nullptr;
}

// Bracket for work on a caller's stream that rewrites replicas or the hot set with plain stores (the
// flag-driven merge, nups_set_management): it must not overlap a background merge.  `begin` keeps the
// thread from enqueueing and orders the work after the last background merge; `end` orders later
// background merges after the work.
void nups_background_begin(nups_store* s, cudaStream_t st)
{
    nups_background* bg = s->bg;
    if (!bg) return;
    bg->mu.lock();
    if (bg->any_merge) cudaStreamWaitEvent(st, bg->merged, 0);
}

void nups_background_end(nups_store* s, cudaStream_t st)
{
    nups_background* bg = s->bg;
    if (!bg) return;
    if (cudaEventRecord(bg->fence, st) == cudaSuccess) cudaStreamWaitEvent(bg->stream, bg->fence, 0);
    bg->mu.unlock();
}

uint64_t nups_background_merges(nups_store* s)
{
    nups_background* bg = s->bg;
    if (!bg) return 0;
    std::lock_guard<std::mutex> g(bg->mu);
    return bg->merges;
}

extern "C" nups_status nups_set_sync_period(nups_store* s, uint32_t period_us)
{
    if (!s) return NUPS_EINVAL;
    if (period_us && s->cfg.deterministic) return NUPS_ESTATE;     // merges at arbitrary times are not reproducible
    if (period_us && (s->vb != 4 || s->cfg.merge_mean)) return NUPS_ESTATE;   // the background merge moves fp32 sums only
    if (!s->bg) {
        if (period_us == 0) return NUPS_OK;
        return nups_background_start(s, period_us);
    }
    {
        std::lock_guard<std::mutex> g(s->bg->mu);
        s->bg->period_us = period_us;
    }
    s->bg->cv.notify_all();
    if (period_us == 0) CK(cudaStreamSynchronize(s->bg->stream));  // merges already enqueued are done on return
    return NUPS_OK;
}
