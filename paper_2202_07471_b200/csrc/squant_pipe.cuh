// Pipelined kernel for layers of long 3x3 channels (more than 8192 weights per output channel).
//
// The grouped kernel runs one channel per CTA from start to end, and the chain of its phases -
// wait for the staged channel, absmax, SQuant-E/K, channel sum, SQuant-C, stores - is what bounds
// it: while a CTA waits, its warps issue nothing.  Here ONE persistent CTA per SM keeps two
// channels in flight, in two complete sets of buffers, and three kinds of warps work on them at
// the same time:
//   copy warp (one thread)    fetches channel c + 2 by a bulk asynchronous copy as soon as the
//                             staged weights of channel c are dead; it also hands out the work
//   16 quantizer warps        absmax, scale, SQuant-E, SQuant-K and the candidates of channel c + 1
//   4 finisher warps          exact redo, SQuant-C and the stores of channel c
// They meet only through mbarriers (full / weights-free / quantized / buffers-free, one of each
// per buffer set); every wait on them is bounded, and a wait that runs out is recorded in the
// device status word while the thread carries on (the outputs of that launch are then
// incomplete, the kernel still ends).
//
// Channels are handed out dynamically: CTA b starts with channel b, every further one is drawn
// from a counter in device memory.  The last CTA to leave puts the counter back to zero, so every
// launch finds it clean.
#pragma once

#include "squant_device.cuh"

namespace sq {

constexpr int kPipeQuantThreads = 512;
constexpr int kPipeFinThreads = 128;
constexpr int kPipeThreads = kPipeQuantThreads + kPipeFinThreads + 32;
constexpr int kPipeCtrlBytes = 256;
constexpr int kPipeScratchBytes = 4 * kHistBins + 256;   // histogram + reduction area at the end of a set

// Work counters, one slot per launch plan.  Launches that share a slot must not overlap; a slot
// belongs to one plan, i.e. to one set of output buffers, for which overlapping launches would
// race on the outputs anyway.
constexpr int kTicketSlots = 1024;
__device__ unsigned g_ticket[kTicketSlots];
__device__ unsigned g_done[kTicketSlots];

// Control block behind the two buffer sets.
struct PipeCtrl {
    unsigned long long full[2];    // the staged weights of the set have arrived (copy warp -> quantizers)
    unsigned long long wfree[2];   // the staged weights are dead (finishers -> copy warp)
    unsigned long long qdone[2];   // codes, candidates, histogram, sums are complete (quantizers -> finishers)
    unsigned long long afree[2];   // the set's buffers may be rewritten (finishers -> quantizers)
    int ring[2];                   // channel (item) being staged into the set, -1: no more work (copy warp -> quantizers)
    int fitem[2];                  // the same, handed on by the quantizers: the copy warp may already have
                                   // written the set's next channel into ring[] when the finishers start
    unsigned amax[3];              // absmax accumulators, rotating
    float scale[2];                // the channel's scale, for the finishers
    int abort;                     // a wait ran out: nobody waits any more (the launch's outputs are void)
};
static_assert(sizeof(PipeCtrl) <= kPipeCtrlBytes, "control block too large");

// Bounded wait.  After the first wait of the CTA that ran out, all waits return at once: the
// kernel then runs through its remaining channels without synchronisation (every index it
// forms is bounded whatever the data) and ends; the status word tells the host.
__device__ __forceinline__ void pipe_wait(PipeCtrl *ctrl, void *bar, unsigned parity)
{
    if (*reinterpret_cast<volatile int *>(&ctrl->abort)) return;
    if (!mbar_wait(bar, parity)) {
        *reinterpret_cast<volatile int *>(&ctrl->abort) = 1;
        atomicExch(&g_device_status, 1);
    }
}

// Lane 0 of the warp waits, the others wait for lane 0.
__device__ __forceinline__ void pipe_wait_warp(PipeCtrl *ctrl, void *bar, unsigned parity)
{
    if ((threadIdx.x & 31) == 0) pipe_wait(ctrl, bar, parity);
    __syncwarp();
}

__device__ __forceinline__ int pipe_layer_of(const LaunchTable &tbl, int item)
{
    int layer = 0;   // last layer whose first item is <= item
#pragma unroll 1
    for (int step = tbl.top_step; step > 0; step >>= 1)
        if (layer + step < tbl.n_layers && tbl.first_item[layer + step] <= item) layer += step;
    return layer;
}

// SQuant-E/K and candidates of one channel by the plain IEEE division, one thread per kernel: for
// channels whose scale is outside the range of the reciprocal sequence.  Fills the same buffers
// as k9_quantize (no kernel is left for the exact redo).
__device__ __forceinline__ long long k9_quantize_div(const LayerDesc &L, int m, const Group &G,
                                                     unsigned char *slice, float s)
{
    const int N = L.N;
    const float *wbuf = reinterpret_cast<const float *>(slice);
    unsigned char *cbuf = slice + L.off_codes;
    int *ev = reinterpret_cast<int *>(slice + L.off_ev);
    int *vv = reinterpret_cast<int *>(slice + L.off_vv);
    unsigned char *vi = slice + L.off_vi;
    int *hist = reinterpret_cast<int *>(slice + L.off_hist);
    float *kerr = L.kerr ? L.kerr + static_cast<size_t>(m) * N : nullptr;
    long long esum = 0;
    for (int n = G.t; n < N; n += G.g) {
        const KernelOut o = kernel9_exact_t<true>(wbuf + n * 9, s, 0.0f, cbuf + n * 9);
        ev[n] = o.e;
        vv[n] = o.v;
        vi[n] = static_cast<unsigned char>(o.idx);
        if (kerr) kerr[n] = __fmul_rn(__int2float_rn(o.e), 0x1p-30f);
        if (o.v != 0) hist_add(hist, o.v);
        esum += o.e;
    }
    return esum;
}

// Layers: 3x3, N a multiple of 4, SQuant-K on; every layer
// descriptor carries the 512-thread layout of the grouped kernel, and a buffer set is one such
// slice (set_stride bytes apart).  One item = one output channel.
__global__ void __launch_bounds__(kPipeThreads, 1)
squant_pipe_kernel(const __grid_constant__ LaunchTable tbl, int qmax, unsigned mode, int n_items, int slot,
                   int set_stride)
{
    extern __shared__ __align__(16) unsigned char smem[];
    PipeCtrl *ctrl = reinterpret_cast<PipeCtrl *>(smem + 2 * static_cast<size_t>(set_stride));
    const int tid = threadIdx.x;
    // In every layer of the launch the channel-step scratch (histogram, then the reduction area)
    // is the last kPipeScratchBytes of a set: it can be cleared without knowing the layer.
    const int hist_off = set_stride - kPipeScratchBytes, red_off = hist_off + 4 * kHistBins;
    if (tid < kPipeCtrlBytes / 4) reinterpret_cast<int *>(ctrl)[tid] = 0;
    for (int j = tid; j < 2 * (kPipeScratchBytes / 4); j += kPipeThreads) {
        const int b = j / (kPipeScratchBytes / 4), k = j % (kPipeScratchBytes / 4);
        reinterpret_cast<int *>(smem + static_cast<size_t>(b) * set_stride + hist_off)[k] = 0;
    }
    __syncthreads();
    if (tid == 0) {
        for (int b = 0; b < 2; ++b) {
            mbar_init(&ctrl->full[b], 1);
            mbar_init(&ctrl->wfree[b], 1);
            mbar_init(&ctrl->qdone[b], kPipeQuantThreads / 32);
            mbar_init(&ctrl->afree[b], 1);
        }
    }
    __syncthreads();

    if (tid >= kPipeQuantThreads + kPipeFinThreads) {
        // ---------------------------------------------------------------- copy warp
        if (tid != kPipeQuantThreads + kPipeFinThreads) return;
        int issued = 0;   // copies issued so far
        for (int i = 0;; ++i) {
            const int b = i & 1, u = i >> 1;
            int item = blockIdx.x;   // the grid never exceeds the number of items
            if (i > 0) {
                const unsigned t = gridDim.x + atomicAdd(&g_ticket[slot], 1u);
                item = t < static_cast<unsigned>(n_items) ? static_cast<int>(t) : -1;
            }
            if (u >= 1) {
                // The set's staged weights are dead once its quantizers are done, unless kernels
                // wait for the exact redo: then the finishers say when.  (Skipping the second
                // wait is safe: the finishers still arrive once per channel, and a later wait
                // names the phase it needs.)
                const unsigned par = static_cast<unsigned>(u - 1) & 1u;
                pipe_wait(ctrl, &ctrl->qdone[b], par);
                const int redo = reinterpret_cast<const volatile int *>(smem + static_cast<size_t>(b) * set_stride + red_off + 128)[6];
                if (redo != 0) pipe_wait(ctrl, &ctrl->wfree[b], par);
            }
            // after a wait of this CTA has run out, no further channel is started: the end mark goes out
            if (*reinterpret_cast<volatile int *>(&ctrl->abort)) item = -1;
            ctrl->ring[b] = item;
            if (item < 0) {
                mbar_arrive(&ctrl->full[b]);
                break;
            }
            const int layer = pipe_layer_of(tbl, item);
            const LayerDesc &L = tbl.layers[layer];
            const float *wg = L.w + static_cast<size_t>(item - tbl.first_item[layer]) * L.NK;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the set's earlier readers before the async write
            bulk_load(smem + static_cast<size_t>(b) * set_stride, wg, static_cast<unsigned>(L.NK) * 4u, &ctrl->full[b]);
            issued = i + 1;
        }
        if (*reinterpret_cast<volatile int *>(&ctrl->abort)) {
            // leaving after a wait ran out: the last two copies may still be in flight into this
            // CTA's shared memory; wait for them (bounded) before the CTA may end
            for (int j = max(issued - 2, 0); j < issued; ++j) mbar_wait(&ctrl->full[j & 1], static_cast<unsigned>(j >> 1) & 1u);
        }
        // every ticket this CTA draws has been drawn: the last CTA to get here resets the slot
        __threadfence();
        if (atomicAdd(&g_done[slot], 1u) == gridDim.x - 1) {
            g_ticket[slot] = 0;
            g_done[slot] = 0;
            __threadfence();
        }
        return;
    }

    if (tid < kPipeQuantThreads) {
        // ---------------------------------------------------------------- quantizer warps
        Group G;
        G.g = kPipeQuantThreads;
        G.t = tid;
        G.bar = 1;
        for (int i = 0;; ++i) {
            const int b = i & 1, u = i >> 1;
            pipe_wait_warp(ctrl, &ctrl->full[b], static_cast<unsigned>(u) & 1u);
            const int item = ctrl->ring[b];
            if (item < 0) {   // pass the end on to the finishers (once they are done with the set's last channel)
                if (u >= 1) pipe_wait_warp(ctrl, &ctrl->afree[b], static_cast<unsigned>(u - 1) & 1u);
                if (tid == 0) ctrl->fitem[b] = -1;
                G.sync();
                if ((tid & 31) == 0) mbar_arrive(&ctrl->qdone[b]);
                break;
            }
            const int layer = pipe_layer_of(tbl, item);
            const LayerDesc &L = tbl.layers[layer];
            const int m = item - tbl.first_item[layer];
            unsigned char *slice = smem + static_cast<size_t>(b) * set_stride;
            if (tid == 0) ctrl->amax[(i + 1) % 3] = 0u;   // the next channel's accumulator: idle since two barriers ago
            float amax = 0.0f;
            {
                const int nv = L.NK >> 2;
                const float4 *src = reinterpret_cast<const float4 *>(slice);
#pragma unroll 3
                for (int j = tid; j < nv; j += kPipeQuantThreads) {
                    const float4 t = src[j];
                    amax = fmaxf(fmaxf(amax, fabsf(t.x)), fmaxf(fabsf(t.y), fmaxf(fabsf(t.z), fabsf(t.w))));
                }
            }
            const unsigned wmax = __reduce_max_sync(kFull, __float_as_uint(amax));   // >= 0: uint order = float order
            if ((tid & 31) == 0) atomicMax(&ctrl->amax[i % 3], wmax);
            // From here on the set's other buffers are needed (the finishers have cleared the
            // scratch): the first thread makes sure of it on behalf of all, before the barrier.
            if (tid == 0 && u >= 1) pipe_wait(ctrl, &ctrl->afree[b], static_cast<unsigned>(u - 1) & 1u);
            G.sync();
            amax = __uint_as_float(ctrl->amax[i % 3]);
            const float s = (amax < 0x1p-100f) ? 1.0f : __fdiv_rn(amax, static_cast<float>(qmax));
            if (tid == 0) {
                ctrl->scale[b] = s;
                ctrl->fitem[b] = item;
            }
            long long esum;
            if (s >= 0x1p-60f && s <= 0x1p60f) {
                const float s2 = __fmul_rn(s, 0x1p-30f);
                esum = k9_quantize(L, m, G, slice, s, s2, __frcp_rn(s2));
            } else {
                esum = k9_quantize_div(L, m, G, slice, s);
            }
            {   // channel sum: two 32-bit warp reductions, one shared atomic per warp
                const int hi = __reduce_add_sync(kFull, static_cast<int>(esum >> 16));
                const int lo = __reduce_add_sync(kFull, static_cast<int>(esum & 0xffff));
                if ((tid & 31) == 0)
                    atomicAdd(reinterpret_cast<unsigned long long *>(slice + L.off_red + 208),
                              static_cast<unsigned long long>((static_cast<long long>(hi) << 16) + lo));
            }
            __syncwarp();
            if ((tid & 31) == 0) mbar_arrive(&ctrl->qdone[b]);
        }
        return;
    }

    // -------------------------------------------------------------------- finisher warps
    Group G;
    G.g = kPipeFinThreads;
    G.t = tid - kPipeQuantThreads;
    G.bar = 2;
    for (int i = 0;; ++i) {
        const int b = i & 1, u = i >> 1;
        pipe_wait_warp(ctrl, &ctrl->qdone[b], static_cast<unsigned>(u) & 1u);
        const int item = ctrl->fitem[b];
        if (item < 0) break;
        const int layer = pipe_layer_of(tbl, item);
        const LayerDesc &L = tbl.layers[layer];
        const int m = item - tbl.first_item[layer];
        unsigned char *slice = smem + static_cast<size_t>(b) * set_stride;
        const float s = ctrl->scale[b];
        const float s2 = __fmul_rn(s, 0x1p-30f);
        const float y = __frcp_rn(s2);   // only the exact redo uses it (fast-path channels)
        float *kerr = L.kerr ? L.kerr + static_cast<size_t>(m) * L.N : nullptr;
        // packed rows are put together in the set's candidate arrays (dead by then): the staged
        // weights' place may already be receiving the set's next channel
        finish_channel_hist<9>(L, m, G, slice, s, mode, 0ll, kerr, y, s2, &ctrl->wfree[b], slice + L.off_ev);
        G.sync();   // every finisher is done with the set; the first one has waited for its bulk store
        {   // leave the channel-step scratch cleared for the set's next channel
            int *scratch = reinterpret_cast<int *>(slice + hist_off);
            for (int j = G.t; j < kHistBins; j += kPipeFinThreads) scratch[j] = 0;
            if (G.t == 0) {
                unsigned char *red = slice + red_off;
                reinterpret_cast<int *>(red + 128)[5] = 0;                    // boundary-list count
                reinterpret_cast<int *>(red + 128)[6] = 0;                    // redo-list count
                *reinterpret_cast<unsigned long long *>(red + 208) = 0ull;   // channel-sum accumulator
            }
        }
        G.sync();
        if (G.t == 0) mbar_arrive(&ctrl->afree[b]);
    }
}

}  // namespace sq
