// Streaming kernel for layers of long 3x3 channels with plain int8 codes (no packed, no
// dequantized output): the successor of the pipelined kernel on its most common case.
//
// In the pipelined kernel the quantizer warps of an SM walk through a channel's phases together
// (wait, absmax, barrier, SQuant-E/K, sum) and four finisher warps run SQuant-C as a chain of
// short barrier-separated steps over per-kernel arrays in shared memory; both chains are about
// as long as the whole period, so neither can be shortened alone.  A chain of dependent
// instructions is what costs here (twenty and more cycles per instruction beside fifteen busy
// warps), so this kernel keeps the quantizer warps' step down to straight, independent work and
// as few hand-overs as the method allows:
//
//   copy warp (one thread)   fetches channel c + 2 by a bulk asynchronous copy as soon as every
//                            quantizer warp has read the weights of channel c; hands out the work
//   two scale warps          absmax of the staged channel (a pass over its weights in shared memory
//                            that the quantizers need not make), then its scale, once for all
//   16 quantizer warps       step c: SQuant-E on the thread's 36 weights, SQuant-K and Algorithm 3
//                            on its four kernels, then SQuant-C's flips on its four kernels of
//                            channel c - 1 (one comparison tells a thread whether any of them is
//                            concerned, so the channel step needs no pass over per-kernel arrays)
//   channel warp             channel sum -> flip count -> scan of the candidate histogram ->
//                            thresholds (published to the quantizers); one step later the exact
//                            ranking of the few candidates inside the boundary bin, the bulk store
//                            of the codes, scale and channel error
//
// Two buffers for staged weights, four for codes (a channel's codes stay in shared memory until
// the channel warp has stored them, up to two steps after they were written; four buffers make
// "the buffer is free again" follow from waits the quantizers make anyway).  The quantizer warps
// never meet at a barrier.  The roles meet through mbarriers only - per step a quantizer warp
// waits for two (scale ready, decision published; both normally complete long before) and
// arrives at two; every wait is bounded, and a wait that runs out is recorded in the device
// status word while the CTA stops taking work (the outputs of that launch are then incomplete,
// the kernel still ends).
//
// Registers are the scarce resource (twenty warps: 96 per thread, and a spilled value comes back
// from L2 here, the L1 being all shared memory), which shaped two things: what SQuant-C needs
// of a thread's kernels one step later waits in a scratch area in global memory instead of in
// registers (a dozen kernels in two thousand are flipped; the others' data is never read back),
// and the four kernels of a thread are settled one after the other.
#pragma once

#include <cstddef>

#include "squant_pipe.cuh"

namespace sq {

constexpr int kStreamQuantWarps = 16;
constexpr int kStreamQuantThreads = 32 * kStreamQuantWarps;
constexpr int kStreamHelpThreads = 128;                     // channel warp, copy warp, two scale warps: the CTA's first
                                                            // four warps, one per scheduler
constexpr int kStreamThreads = kStreamHelpThreads + kStreamQuantThreads;
constexpr int kStreamListCap = 128;                        // candidates ranked exactly inside the boundary bin
constexpr int kStreamQueueCap = 128;                       // quantizer threads per channel that hand their flips to the channel warp
constexpr int kStreamCtrlBytes = 3328;

// SQuant-C of one channel as the quantizers need it (sixteen bytes, read as one word).
struct StreamDecision {
    int kind;       // 0: no flips, 1: thresholds on v * sgn_c, 2: threshold on the 48-bit key, 3: one more digit of the
                    //    key is wanted first: count the candidates that share the digits fixed so far
    int sgn_c;      // direction of the flips
    int t_all;      // kind 1: candidates with v * sgn_c >= t_all are flipped outright; kind 3: bit position of the digit
    int t_list;     //         those in [t_list, t_all) are listed for the exact ranking
};

struct StreamListEntry {
    int a;      // v * sgn_c
    int n;      // kernel
    int pos;    // byte of the candidate's code inside the channel
    int e;      // the kernel's error sum before the flip
};

// A staged channel as the copy thread describes it to the others.
struct StreamSlot {
    int item;    // -1: no more work
    int layer;   // index into the launch table
    int m;       // output channel inside the layer
    int quads;   // N / 4: threads with kernels
    float *kerr; // the channel's row of kernel sums in global memory, or null
    long long pad;
};

struct StreamCtrl {
    unsigned long long full[2];      // staged weights have arrived (copy -> quantizers)
    unsigned long long wread[2];     // every quantizer warp has the channel's weights in registers (quantizers -> copy)
    unsigned long long sready[2];    // the channel's scale is published (scale warp -> quantizers)
    unsigned long long qdone[2];     // codes, histogram, sums of the step complete, the previous channel's flips applied
                                     // (quantizers -> channel warp)
    unsigned long long cdec[2];      // decision published (channel warp -> quantizers)
    unsigned long long hand[2];      // every quantizer warp has added its candidates to the digit histogram (rare)
    unsigned long long cdec2[2];     // next decision of a digit-by-digit selection
    unsigned long long adone[2];     // both scale warps have put in their half of the channel's absmax
    unsigned long long T[2];         // kind 2: kernels whose candidate key is >= T are flipped; kind 3: digits fixed so far
    unsigned long long acc[2];       // channel sum accumulators
    float *kprev[4];                 // the channel's row of kernel sums, for the flips one step later (by step modulo
                                     // four: a warp still at its flips must not find the next but one step's row)
    __align__(16) StreamDecision dec[2];
    __align__(16) StreamSlot slot[2];
    __align__(16) float4 sc[2];      // s, s * 2^-30, its reciprocal, 1 if the reciprocal sequence applies else 0
    __align__(16) int4 fin[2];       // item (-1: end), layer, channel and scale bits of the step, handed on by the
                                     // quantizers to the channel warp
    int lcount[2];                   // entries in the boundary list
    int qcount[2];                   // entries in the queue of concerned threads
    unsigned short queue[2][kStreamQueueCap];   // quantizer threads with kernels to flip (or to rank)
    int abort;                       // a wait ran out: nobody waits any more
    unsigned amax[2];                // absmax of the staged channel (bit pattern), from the two scale warps
    int scratch[kStreamQuantWarps][12];                // nine words per quantizer warp for the exact routine
    int dummy[kStreamQuantWarps][12];                  // where lanes without kernels put their (void) code bytes
};
static_assert(sizeof(StreamCtrl) <= kStreamCtrlBytes, "control block too large");

// Shared-memory layout of a launch: every layer of it uses the layout of the longest channel.
struct StreamLayout {
    int w_bytes, c_bytes;   // one weight buffer, one codes buffer
    int off_codes, off_hist, off_list, off_ctrl, total;
};

__host__ __device__ inline StreamLayout stream_layout(int nk_max, int n_max)
{
    StreamLayout l;
    l.w_bytes = (4 * nk_max + 15) & ~15;
    l.c_bytes = (nk_max + 15) & ~15;
    l.off_codes = 2 * l.w_bytes;
    (void)n_max;
    l.off_hist = l.off_codes + 4 * l.c_bytes;
    l.off_list = l.off_hist + 2 * 4 * kHistBins;
    l.off_ctrl = l.off_list + 2 * kStreamListCap * static_cast<int>(sizeof(StreamListEntry));
    l.total = l.off_ctrl + kStreamCtrlBytes;
    return l;
}

// Bounded wait, called by whole warps (every lane polls: no divergence, no warp barrier) or by
// single threads.  The common case - the phase is complete - is one try_wait.
__device__ __forceinline__ void stream_wait(StreamCtrl *ctrl, void *bar, unsigned parity)
{
    if (mbar_wait(bar, parity, 1)) return;
    if (*reinterpret_cast<volatile int *>(&ctrl->abort)) return;
    if (!mbar_wait(bar, parity)) {
        *reinterpret_cast<volatile int *>(&ctrl->abort) = 1;
        atomicExch(&g_device_status, 1);
    }
}

// Exact SQuant-K + Algorithm 3 on one 3x3 kernel whose integer perturbations (2^-30 units) sit in
// nine words of shared memory at P and whose SQuant-E code bytes sit at cb.  For the few kernels
// the straight-line selection cannot settle: loops over shared memory, so that it costs the
// common path neither registers nor much code.
__device__ __noinline__ KernelOut kernel9_exact_smem(int *P, unsigned char *cb)
{
    long long e = 0;
#pragma unroll 1
    for (int i = 0; i < 9; ++i) e += P[i];
    int v = 0, idx = 0;
    if (e != 0) {
        const int sgn = e > 0 ? 1 : -1;
        const long long abs_e = e > 0 ? e : -e;
        const int k = flip_count(abs_e);
        int flips = 0, last = -1, cand = -1;
#pragma unroll 1
        for (int r = 0; r <= k; ++r) {
            int best = 0, bi = -1;
#pragma unroll 1
            for (int i = 0; i < 9; ++i) {
                const int key = sgn * P[i];
                if (key > best) { best = key; bi = i; }
            }
            if (bi < 0) break;
            if (r < k) {   // a flipped element changes sign and leaves the candidates by itself
                P[bi] -= sgn * kOne;
                cb[bi] = static_cast<unsigned char>(cb[bi] - sgn);
                last = bi;
                ++flips;
            } else {
                cand = bi;
            }
        }
        e -= static_cast<long long>(sgn) * flips * kOne;
        const int pick = (static_cast<long long>(flips) * kOne > abs_e) ? last : cand;
        if (pick >= 0) {
            idx = pick;
            v = P[pick];
        }
    }
    KernelOut o;
    o.e = static_cast<int>(e);
    o.v = v;
    o.idx = idx;
    return o;
}

// What SQuant-C needs of a quantizer thread's four kernels once their channel is decided - error sums,
// candidates, positions - waits in a scratch area in global memory (registers are what this kernel is
// short of, and the flips are few: a dozen kernels in two thousand).  The thread itself keeps the
// largest and the smallest candidate, which tell it whether any of its kernels is concerned at all.
// Per CTA and set: 512 x int4 sums, 512 x int4 candidates, 512 x 4 index bytes.
constexpr int kStreamHeldBytes = kStreamQuantThreads * 36;   // one set
constexpr int kStreamHeldSets = 4;   // by step modulo four, like the code buffers: a set is rewritten only after a wait
                                     // that implies the channel warp is done with it
struct StreamHeld {
    int vmax, vmin;   // largest and smallest of the four candidates (0 where there are no kernels)
    bool have;        // a previous channel exists
};

// SQuant-K and Algorithm 3 on kernel KQ of the thread's quad: perturbations P2 (pairs, already
// normalised to the sign of the kernel's float sum ef), code bytes at cq + 9 KQ.  Straight-line;
// returns true for a kernel the selection cannot settle (its staged codes are then untouched).
template <int KQ>
__device__ __forceinline__ bool stream_kernel(const float2 (&P2)[18], float ef, unsigned char *cq,
                                              int &e_out, int &v_out, unsigned &idx_out)
{
    float Pk[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) {
        const int el = 9 * KQ + i;
        Pk[i] = (el & 1) ? P2[el >> 1].y : P2[el >> 1].x;
    }
    return kernel9_select(Pk, ef, cq + 9 * KQ, e_out, v_out, idx_out);
}

// The kernels stream_kernel<KQ> reported (about one in 10^5 on random weights): settled exactly,
// one lane after the other on the warp's scratch words.  Called by the whole warp.
template <int KQ>
__device__ __forceinline__ void stream_rare(bool rare, const float2 (&P2)[18], float ef, unsigned char *cq, int *scr,
                                            int &e_out, int &v_out, unsigned &idx_out)
{
    const unsigned rm = __ballot_sync(kFull, rare);
    const int g = (__float_as_int(ef) >> 31) | 1;
    for (unsigned left = rm; left != 0u; left &= left - 1u) {
        if (static_cast<int>(threadIdx.x & 31u) == __ffs(left) - 1) {
#pragma unroll
            for (int i = 0; i < 9; ++i) {
                const int el = 9 * KQ + i;
                scr[i] = g * __float2int_rn((el & 1) ? P2[el >> 1].y : P2[el >> 1].x);
            }
            const KernelOut x = kernel9_exact_smem(scr, cq + 9 * KQ);
            e_out = x.e;
            v_out = x.v;
            idx_out = static_cast<unsigned>(x.idx);
        }
        __syncwarp();
    }
}

// SQuant-C's flips on the four kernels of quantizer thread t, whose details wait in the scratch set at
// hset: kernels above the threshold are flipped here (code byte in the channel's staged codes, error sum
// in global memory), members of the boundary bin go to the list for the exact ranking.
__device__ __forceinline__ void stream_flip_thread(int t, const StreamDecision &D, unsigned long long T,
                                                   const unsigned char *hset, unsigned char *codes, float *kerr_row,
                                                   StreamListEntry *blist, int *lcount)
{
    SQ_DBG(t >= 0 && t < kStreamQuantThreads, 21);   // a quantizer thread's index
    // (written by another thread of this CTA two hand-overs ago: read past the L1)
    const int4 he = __ldcg(reinterpret_cast<const int4 *>(hset) + t);
    const int4 hv = __ldcg(reinterpret_cast<const int4 *>(hset + 16 * kStreamQuantThreads) + t);
    const unsigned hidx = __ldcg(reinterpret_cast<const unsigned *>(hset + 32 * kStreamQuantThreads) + t);
    const int hvv[4] = {hv.x, hv.y, hv.z, hv.w}, hee[4] = {he.x, he.y, he.z, he.w};
    const int sgn_c = D.sgn_c;
    const int t_min = D.kind == 2 ? 1 : min(D.t_all, D.t_list);
#pragma unroll
    for (int kq = 0; kq < 4; ++kq) {
        const int a = hvv[kq] * sgn_c;
        if (a >= t_min) {
            const int n = 4 * t + kq;
            SQ_DBG(((hidx >> (8 * kq)) & 15u) < 9u, 22);   // the candidate is one of the kernel's nine elements
            const int pos = 36 * t + 9 * kq + min(static_cast<int>((hidx >> (8 * kq)) & 15u), 8);
            bool take;
            if (D.kind == 2) {
                take = cand_key(hvv[kq], sgn_c, n) >= T;
            } else {
                take = a >= D.t_all;
                if (!take) {
                    const int at = atomicAdd(lcount, 1);
                    if (at < kStreamListCap) {
                        StreamListEntry en;
                        en.a = a;
                        en.n = n;
                        en.pos = pos;
                        en.e = hee[kq];
                        blist[at] = en;
                    }
                }
            }
            if (take) {
                codes[pos] = static_cast<unsigned char>(codes[pos] - sgn_c);
                if (kerr_row) kerr_row[n] = __fmul_rn(__int2float_rn(hee[kq] - sgn_c * kOne), 0x1p-30f);
            }
        }
    }
}

// One warp over 256 counts, highest bins first: lane l holds bins 8 (31 - l) .. 8 (31 - l) + 7 in c[0..7].
// Finds the bin in which the want-th largest entry falls, want = min(kc, total): its index, its
// count and how many of its entries are among the want largest.  Returns want (0: nothing there).
__device__ __forceinline__ int stream_boundary(const int (&c)[8], int lane, int kc, int &bb, int &cnt, int &rem)
{
    const int grp = 31 - lane;
    const int s8 = ((c[0] + c[1]) + (c[2] + c[3])) + ((c[4] + c[5]) + (c[6] + c[7]));
    int incl = s8;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += t;
    }
    const int total = __shfl_sync(kFull, incl, 31);
    const int want = min(kc, total);
    if (want <= 0) return 0;
    const int src = __ffs(__ballot_sync(kFull, incl >= want)) - 1;   // the lane holding the boundary bin
    int b1 = 0, c1 = 0, cum = incl - s8;
    bool found = false;
#pragma unroll
    for (int q = 7; q >= 0; --q) {
        if (!found) {
            if (cum + c[q] >= want) { b1 = grp * 8 + q; c1 = c[q]; found = true; }
            else cum += c[q];
        }
    }
    bb = __shfl_sync(kFull, b1, src);
    cnt = __shfl_sync(kFull, c1, src);
    rem = want - __shfl_sync(kFull, cum, src);
    return want;
}

// Layers: 3x3, N a multiple of 4 and at most 4 * 512, SQuant-K on, absmax scales, int8 codes only.
// One item = one output channel; nk_max / n_max are the longest channel of the launch (weights /
// kernels), from which every CTA derives the same layout.
__global__ void __launch_bounds__(kStreamThreads, 1)
squant_stream_kernel(const __grid_constant__ LaunchTable tbl, int qmax, unsigned mode, int n_items, int slot,
                     int nk_max, int n_max, unsigned char *held_scratch)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const StreamLayout lay = stream_layout(nk_max, n_max);
    StreamCtrl *ctrl = reinterpret_cast<StreamCtrl *>(smem + lay.off_ctrl);
    const int tid = threadIdx.x;
    for (int j = tid; j < kStreamCtrlBytes / 4; j += kStreamThreads) reinterpret_cast<int *>(ctrl)[j] = 0;
    for (int j = tid; j < 2 * kHistBins; j += kStreamThreads) reinterpret_cast<int *>(smem + lay.off_hist)[j] = 0;
    __syncthreads();
    if (tid == 0) {
        for (int b = 0; b < 2; ++b) {
            mbar_init(&ctrl->full[b], 1);
            mbar_init(&ctrl->wread[b], kStreamQuantWarps);
            mbar_init(&ctrl->sready[b], 1);
            mbar_init(&ctrl->qdone[b], kStreamQuantWarps);
            mbar_init(&ctrl->cdec[b], 1);
            mbar_init(&ctrl->hand[b], kStreamQuantWarps);
            mbar_init(&ctrl->cdec2[b], 1);
            mbar_init(&ctrl->adone[b], 2);
        }
    }
    __syncthreads();

    if (tid >= 32 && tid < 64) {
        // ---------------------------------------------------------------- copy warp
        if (tid != 32) return;
        int issued = 0;            // copies issued so far
        int item = blockIdx.x;     // the grid never exceeds the number of items
        bool ended = false;        // the end mark has gone out
        // stages the next channel (or the end mark) into weight buffer b
        auto stage = [&](int b) {
            // after a wait of this CTA has run out, no further channel is started
            if (*reinterpret_cast<volatile int *>(&ctrl->abort)) item = -1;
            StreamSlot sl;
            sl.item = item; sl.layer = 0; sl.m = 0; sl.quads = 0; sl.kerr = nullptr; sl.pad = 0;
            if (item < 0) {
                ctrl->slot[b] = sl;
                mbar_arrive(&ctrl->full[b]);
                ended = true;
                return;
            }
            sl.layer = pipe_layer_of(tbl, item);
            const LayerDesc &L = tbl.layers[sl.layer];
            sl.m = item - tbl.first_item[sl.layer];
            sl.quads = L.N >> 2;
            sl.kerr = L.kerr ? L.kerr + static_cast<size_t>(sl.m) * L.N : nullptr;
            ctrl->slot[b] = sl;
            const float *wg = L.w + static_cast<size_t>(sl.m) * L.NK;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the buffer's earlier readers before the async write
            bulk_load(smem + static_cast<size_t>(b) * lay.w_bytes, wg, static_cast<unsigned>(L.NK) * 4u, &ctrl->full[b]);
            ++issued;
            // the next channel is drawn now: the counter's latency passes during the waits
            const unsigned t = gridDim.x + atomicAdd(&g_ticket[slot], 1u);
            item = t < static_cast<unsigned>(n_items) ? static_cast<int>(t) : -1;
        };
        stage(0);
        if (!ended) stage(1);
        for (int k = 0; !ended; ++k) {
            // every quantizer warp has channel k in registers: channel k + 2 takes its place
            stream_wait(ctrl, &ctrl->wread[k & 1], static_cast<unsigned>(k >> 1) & 1u);
            stage(k & 1);
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

    if (tid >= 64 && tid < kStreamHelpThreads) {
        // ---------------------------------------------------------------- scale warps
        // absmax of every staged channel (a pass over its weights in shared memory that the
        // quantizer warps need not make), a half each; the first one then derives the scale and
        // what SQuant-E needs of it
        const int lane = tid & 31, half = (tid - 64) >> 5;
        for (int c = 0;; ++c) {
            const int b = c & 1;
            stream_wait(ctrl, &ctrl->full[b], static_cast<unsigned>(c >> 1) & 1u);
            const StreamSlot sl = ctrl->slot[b];
            if (sl.item < 0) {   // the end mark goes on to the quantizers
                if (tid == 64) mbar_arrive(&ctrl->sready[b]);
                break;
            }
            const int nv = 9 * sl.quads, nh = (nv + 1) >> 1;
            const float4 *src = reinterpret_cast<const float4 *>(smem + static_cast<size_t>(b) * lay.w_bytes);
            const int end = half ? nv : nh;
            float a4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            int j = (half ? nh : 0) + lane;
            for (; j + 7 * 32 < end; j += 8 * 32) {   // eight loads in flight
                float4 t[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) t[k] = src[j + 32 * k];
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    a4[k & 3] = fmaxf(fmaxf(a4[k & 3], fabsf(t[k].x)), fmaxf(fabsf(t[k].y), fmaxf(fabsf(t[k].z), fabsf(t[k].w))));
            }
            for (; j < end; j += 32) {
                const float4 t = src[j];
                a4[0] = fmaxf(fmaxf(a4[0], fabsf(t.x)), fmaxf(fabsf(t.y), fmaxf(fabsf(t.z), fabsf(t.w))));
            }
            const unsigned wmax = __reduce_max_sync(kFull, __float_as_uint(fmaxf(fmaxf(a4[0], a4[1]), fmaxf(a4[2], a4[3]))));   // >= 0: uint order = float order
            if (lane == 0) {
                atomicMax(&ctrl->amax[b], wmax);
                mbar_arrive(&ctrl->adone[b]);
            }
            if (tid == 64) {
                stream_wait(ctrl, &ctrl->adone[b], static_cast<unsigned>(c >> 1) & 1u);
                const float amax = __uint_as_float(*reinterpret_cast<volatile unsigned *>(&ctrl->amax[b]));
                ctrl->amax[b] = 0u;   // for the buffer's next channel (staged only after this one's scale is out)
                const float s = (amax < 0x1p-100f) ? 1.0f : __fdiv_rn(amax, static_cast<float>(qmax));
                const bool fast = s >= 0x1p-60f && s <= 0x1p60f;
                const float s2 = fast ? __fmul_rn(s, 0x1p-30f) : 0.0f;
                ctrl->sc[b] = make_float4(s, s2, fast ? __frcp_rn(s2) : 0.0f, fast ? 1.0f : 0.0f);
                mbar_arrive(&ctrl->sready[b]);
            }
            __syncwarp();
        }
        return;
    }

    if (tid >= kStreamHelpThreads) {
        // ---------------------------------------------------------------- quantizer warps
        const int qt = tid - kStreamHelpThreads;   // owns kernels 4 qt .. 4 qt + 3 of every channel
        const int warp = qt >> 5, lane = qt & 31;
        int *scr = ctrl->scratch[warp];
        unsigned hand_par = 0u;   // phases of the hand-over barriers used so far: bit b for set b
        StreamHeld held;
        held.vmax = 0;
        held.vmin = 0;
        held.have = false;
        unsigned char *hs = held_scratch + static_cast<size_t>(blockIdx.x) * (kStreamHeldSets * kStreamHeldBytes);
        auto held_e = [&](int set) { return reinterpret_cast<int4 *>(hs + set * kStreamHeldBytes) + qt; };
        auto held_v = [&](int set) { return reinterpret_cast<int4 *>(hs + set * kStreamHeldBytes + 16 * kStreamQuantThreads) + qt; };
        auto held_i = [&](int set) { return reinterpret_cast<unsigned *>(hs + set * kStreamHeldBytes + 32 * kStreamQuantThreads) + qt; };

        // SQuant-C's flips on the held kernels (channel of set pb, k-th use of the set: parity par)
        auto apply = [&](int pb, unsigned par, int pj) {
            stream_wait(ctrl, &ctrl->cdec[pb], par);
            StreamDecision D = ctrl->dec[pb];
            while (D.kind == 3) {   // warp-uniform (CTA-uniform); at most five rounds
                // A boundary bin too crowded for the list (massive ties): the threshold is found on the
                // 48-bit keys digit by digit, as the general path's radix select does.  The candidates that
                // share the digits fixed so far are counted by the next digit in the channel's (cleared) histogram.
                const int sh = D.t_all;
                const unsigned long long prefix = ctrl->T[pb];
                int *dh = reinterpret_cast<int *>(smem + lay.off_hist) + pb * kHistBins;
                {
                    const int4 hv = *held_v(pj);   // zeros where there are no kernels
                    const int v[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
                    for (int kq = 0; kq < 4; ++kq) {
                        const unsigned long long ck = cand_key(v[kq], D.sgn_c, 4 * qt + kq);
                        if (ck != 0ull && (ck >> (sh + 8)) == prefix) atomicAdd(&dh[static_cast<int>(ck >> sh) & 255], 1);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctrl->hand[pb]);
                stream_wait(ctrl, &ctrl->cdec2[pb], (hand_par >> pb) & 1u);
                hand_par ^= 1u << pb;
                D = ctrl->dec[pb];
            }
            const int t_min = D.kind == 2 ? 1 : min(D.t_all, D.t_list);
            if (D.kind != 0 && (D.sgn_c > 0 ? held.vmax : -held.vmin) >= t_min) {   // rare per thread (v = 0 where there are no kernels)
                // The thread only says that it is concerned: the channel warp, which has the time, looks up the
                // details and does the flips when it completes the channel.  (A queue that is full - a channel
                // with hundreds of flips - leaves the thread to do its own.)
                const int at = atomicAdd(&ctrl->qcount[pb], 1);
                if (at < kStreamQueueCap) {
                    ctrl->queue[pb][at] = static_cast<unsigned short>(qt);
                } else {
                    stream_flip_thread(qt, D, ctrl->T[pb], hs + pj * kStreamHeldBytes,
                                       smem + lay.off_codes + static_cast<size_t>(pj) * lay.c_bytes, ctrl->kprev[pj],
                                       reinterpret_cast<StreamListEntry *>(smem + lay.off_list) + pb * kStreamListCap, &ctrl->lcount[pb]);
                }
            }
        };

        for (int i = 0;; ++i) {
            const int b = i & 1, u = i >> 1, j = i & 3;
            // the channel's scale (the scale warp has been over its weights during the previous step)
            stream_wait(ctrl, &ctrl->sready[b], static_cast<unsigned>(u) & 1u);
            const StreamSlot cur = ctrl->slot[b];
            SQ_DBG(cur.item < n_items && cur.quads >= 0 && cur.quads <= kStreamQuantThreads && cur.layer >= 0 && cur.layer < tbl.n_layers, 24);
            if (cur.item < 0) {
                // the last channel's flips, then the end mark for the channel warp
                if (held.have) apply(b ^ 1, static_cast<unsigned>((i - 1) >> 1) & 1u, (i + 3) & 3);
                if (qt == 0) ctrl->fin[b] = make_int4(-1, 0, 0, 0);
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctrl->qdone[b]);
                break;
            }
            const bool active = qt < cur.quads;
            const unsigned char *wbuf = smem + static_cast<size_t>(b) * lay.w_bytes;
            unsigned char *cq = active ? smem + lay.off_codes + static_cast<size_t>(j) * lay.c_bytes + qt * 36
                                       : reinterpret_cast<unsigned char *>(ctrl->dummy[warp]);
            int *hist = reinterpret_cast<int *>(smem + lay.off_hist) + b * kHistBins;
            float *kerr = cur.kerr ? cur.kerr + 4 * qt : nullptr;
            const float4 sc = ctrl->sc[b];
            if (qt == 0) {
                ctrl->fin[b] = make_int4(cur.item, cur.layer, cur.m, __float_as_int(sc.x));
                ctrl->kprev[j] = cur.kerr;
            }
            int e4[4] = {0, 0, 0, 0}, v4[4] = {0, 0, 0, 0};
            unsigned i4 = 0u;
            if (sc.w != 0.0f) {
                const E2 c2 = make_e2(sc.z, sc.y);
                const float4 *src = reinterpret_cast<const float4 *>(wbuf) + qt * 9;
                unsigned *dst = reinterpret_cast<unsigned *>(cq);
                const float4 z = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                float2 P2[18];   // the quad's 36 perturbations, pair p = elements 2p, 2p + 1
#pragma unroll
                for (int q = 0; q < 9; ++q) {
                    const float4 w = active ? src[q] : z;
                    float2 ta, tb;
                    squant_e_fast2(make_float2(w.x, w.y), c2, ta, P2[2 * q]);
                    squant_e_fast2(make_float2(w.z, w.w), c2, tb, P2[2 * q + 1]);
                    dst[q] = __byte_perm(__byte_perm(__float_as_uint(ta.x), __float_as_uint(ta.y), 0x0040),
                                         __byte_perm(__float_as_uint(tb.x), __float_as_uint(tb.y), 0x0040), 0x5410);
                }
                __syncwarp();   // every lane's weights are in registers: the buffer may be refilled
                if (lane == 0) mbar_arrive(&ctrl->wread[b]);
                // float sums of the four kernels (elements 0-8, 9-17, 18-26, 27-35), for their signs
                float ef[4];
                {
                    const float2 s0 = __fadd2_rn(__fadd2_rn(P2[0], P2[1]), __fadd2_rn(P2[2], P2[3]));
                    const float2 s1 = __fadd2_rn(__fadd2_rn(P2[5], P2[6]), __fadd2_rn(P2[7], P2[8]));
                    const float2 s2p = __fadd2_rn(__fadd2_rn(P2[9], P2[10]), __fadd2_rn(P2[11], P2[12]));
                    const float2 s3 = __fadd2_rn(__fadd2_rn(P2[14], P2[15]), __fadd2_rn(P2[16], P2[17]));
                    ef[0] = __fadd_rn(__fadd_rn(s0.x, s0.y), P2[4].x);
                    ef[1] = __fadd_rn(__fadd_rn(s1.x, s1.y), P2[4].y);
                    ef[2] = __fadd_rn(__fadd_rn(s2p.x, s2p.y), P2[13].x);
                    ef[3] = __fadd_rn(__fadd_rn(s3.x, s3.y), P2[13].y);
                }
                // normalise every perturbation to the sign of its kernel's sum (pairs 4 and 13 straddle two kernels)
                {
                    const float g0 = copysignf(1.0f, ef[0]), g1 = copysignf(1.0f, ef[1]);
                    const float g2 = copysignf(1.0f, ef[2]), g3 = copysignf(1.0f, ef[3]);
                    const float2 G0 = make_float2(g0, g0), G1 = make_float2(g1, g1), G2 = make_float2(g2, g2), G3 = make_float2(g3, g3);
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        P2[p] = __fmul2_rn(P2[p], G0);
                        P2[5 + p] = __fmul2_rn(P2[5 + p], G1);
                        P2[9 + p] = __fmul2_rn(P2[9 + p], G2);
                        P2[14 + p] = __fmul2_rn(P2[14 + p], G3);
                    }
                    P2[4] = __fmul2_rn(P2[4], make_float2(g0, g1));
                    P2[13] = __fmul2_rn(P2[13], make_float2(g2, g3));
                }
                unsigned x0, x1, x2, x3;
                const bool r0 = stream_kernel<0>(P2, ef[0], cq, e4[0], v4[0], x0);
                const bool r1 = stream_kernel<1>(P2, ef[1], cq, e4[1], v4[1], x1);
                const bool r2 = stream_kernel<2>(P2, ef[2], cq, e4[2], v4[2], x2);
                const bool r3 = stream_kernel<3>(P2, ef[3], cq, e4[3], v4[3], x3);
                if (__any_sync(kFull, r0 | r1 | r2 | r3)) {   // one test for the four kernels keeps them in one straight piece of code
                    stream_rare<0>(r0, P2, ef[0], cq, scr, e4[0], v4[0], x0);
                    stream_rare<1>(r1, P2, ef[1], cq, scr, e4[1], v4[1], x1);
                    stream_rare<2>(r2, P2, ef[2], cq, scr, e4[2], v4[2], x2);
                    stream_rare<3>(r3, P2, ef[3], cq, scr, e4[3], v4[3], x3);
                }
                i4 = x0 | (x1 << 8) | (x2 << 16) | (x3 << 24);
            } else {
                // scale outside the range of the reciprocal sequence: plain IEEE division, exact routine
                if (active) {
                    const float *w = reinterpret_cast<const float *>(wbuf) + qt * 36;
#pragma unroll
                    for (int kq = 0; kq < 4; ++kq) {   // unrolled: e4 / v4 must stay in registers
                        const KernelOut o = kernel9_exact_t<true>(w + 9 * kq, sc.x, 0.0f, cq + 9 * kq);
                        e4[kq] = o.e;
                        v4[kq] = o.v;
                        i4 |= static_cast<unsigned>(o.idx) << (8 * kq);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctrl->wread[b]);
            }
            long long esum = 0;
            if (active) {
                esum = static_cast<long long>(e4[0] + e4[1]) + (e4[2] + e4[3]);   // pairs fit 32 bits
                // candidate histogram; |v| < 2^30 for valid input, the mask keeps garbage in range (v = 0 adds nothing)
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    atomicAdd(&hist[(abs(v4[k]) >> 22) & (kHistBins - 1)], v4[k] > 0 ? 1 : ((v4[k] >> 31) & 0x10000));
                if (kerr) {
                    float4 f;
                    f.x = __fmul_rn(__int2float_rn(e4[0]), 0x1p-30f);
                    f.y = __fmul_rn(__int2float_rn(e4[1]), 0x1p-30f);
                    f.z = __fmul_rn(__int2float_rn(e4[2]), 0x1p-30f);
                    f.w = __fmul_rn(__int2float_rn(e4[3]), 0x1p-30f);
                    if ((reinterpret_cast<uintptr_t>(kerr) & 15) == 0) __stcs(reinterpret_cast<float4 *>(kerr), f);
                    else { kerr[0] = f.x; kerr[1] = f.y; kerr[2] = f.z; kerr[3] = f.w; }
                }
            }
            {   // channel sum: two 32-bit warp reductions, one shared atomic per warp
                const int hi = __reduce_add_sync(kFull, static_cast<int>(esum >> 16));
                const int lo = __reduce_add_sync(kFull, static_cast<int>(esum & 0xffff));
                if (lane == 0) atomicAdd(&ctrl->acc[b], static_cast<unsigned long long>((static_cast<long long>(hi) << 16) + lo));
            }
            // SQuant-C's flips on the previous channel's kernels: its decision has been out for most of this step
            if (held.have) apply(b ^ 1, static_cast<unsigned>((i - 1) >> 1) & 1u, (i + 3) & 3);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the codes leave by a bulk copy
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctrl->qdone[b]);
            // what SQuant-C may need of these kernels one step from now (threads without kernels hold zeros)
            *held_e(j) = make_int4(e4[0], e4[1], e4[2], e4[3]);
            *held_v(j) = make_int4(v4[0], v4[1], v4[2], v4[3]);
            *held_i(j) = i4;
            held.vmax = max(max(v4[0], v4[1]), max(v4[2], v4[3]));
            held.vmin = min(min(v4[0], v4[1]), min(v4[2], v4[3]));
            held.have = true;
        }
        return;
    }

    // -------------------------------------------------------------------- channel warp
    // Iteration i starts when the quantizers are done with step i: it decides channel i (the quantizers
    // want that before the end of their next step), then completes channel i - 1, whose flips they
    // applied during step i.
    const int lane = tid;
    unsigned hand_par = 0u;   // phases of the digit-round barriers used so far: bit b for set b
    // channel i - 1, between its decision and its store
    bool p_valid = false, p_listing = false;
    int p_rem = 0, p_sgn = 0, p_m = 0, p_layer = 0;
    long long p_ec = 0;
    float p_s = 0.0f;
    for (int i = 0;; ++i) {
        const int b = i & 1, u = i >> 1;
        stream_wait(ctrl, &ctrl->qdone[b], static_cast<unsigned>(u) & 1u);
        const int4 fin = ctrl->fin[b];
        const int item = fin.x;
        const float s = __int_as_float(fin.w);
        const long long ec = item >= 0 ? static_cast<long long>(ctrl->acc[b]) : 0ll;   // channel sum of step i
        // channel i - 1 as the previous iteration left it
        const bool f_valid = p_valid, f_listing = p_listing;
        const int f_rem = p_rem, f_sgn = p_sgn, f_m = p_m, f_layer = p_layer;
        const long long f_ec = p_ec;
        const float f_s = p_s;
        if (item >= 0) {
            // ---- channel i, SQuant-C: boundary bin of the candidate histogram
            int *hist = reinterpret_cast<int *>(smem + lay.off_hist) + b * kHistBins;
            const int grp = 31 - lane;
            StreamDecision D;
            D.kind = 0; D.sgn_c = 0; D.t_all = 0x7fffffff; D.t_list = 0x7fffffff;
            int rem = 0, k_eff = 0, bb = 0, cnt = 0;
            bool listing = false;
            if ((mode & 4u) && ec != 0) {
                D.sgn_c = ec > 0 ? 1 : -1;
                const int kc = flip_count(ec > 0 ? ec : -ec);
                if (kc > 0) {
                    const int sh = D.sgn_c > 0 ? 0 : 16;   // positive and negative candidates share a word
                    const int4 h0 = reinterpret_cast<const int4 *>(hist)[2 * grp];
                    const int4 h1 = reinterpret_cast<const int4 *>(hist)[2 * grp + 1];
                    const int c[8] = {(h0.x >> sh) & 0xffff, (h0.y >> sh) & 0xffff, (h0.z >> sh) & 0xffff, (h0.w >> sh) & 0xffff,
                                      (h1.x >> sh) & 0xffff, (h1.y >> sh) & 0xffff, (h1.z >> sh) & 0xffff, (h1.w >> sh) & 0xffff};
                    k_eff = stream_boundary(c, lane, kc, bb, cnt, rem);
                    if (k_eff > 0) {
                        if (cnt == rem) {                       // whole boundary bin flipped
                            D.kind = 1;
                            D.t_all = max(bb << 22, 1);         // 0 is "no candidate"
                        } else if (cnt <= kStreamListCap) {     // rank the boundary bin exactly
                            D.kind = 1;
                            D.t_all = (bb + 1) << 22;           // bb + 1 = 256 gives 2^30, above every |v|
                            D.t_list = max(bb << 22, 1);
                            listing = true;
                        } else {                                // crowded bin: further digits of the 48-bit keys
                            D.kind = 3;
                        }
                    }
                }
            }
            // the histogram and the sum are read: leave them cleared for the set's next channel
            reinterpret_cast<int4 *>(hist)[2 * grp] = make_int4(0, 0, 0, 0);
            reinterpret_cast<int4 *>(hist)[2 * grp + 1] = make_int4(0, 0, 0, 0);
            if (D.kind != 3) {
                __syncwarp();
                if (lane == 0) {
                    ctrl->acc[b] = 0ull;
                    ctrl->dec[b] = D;
                    mbar_arrive(&ctrl->cdec[b]);
                }
            } else {
                // The key of a candidate is (|v| << 18) | (2^18 - 1 - kernel): its top eight bits are the bin
                // just found.  Digit by digit (the general path's radix select, with the quantizers doing
                // the counting): ask for the counts of the next digit among the keys that share the digits
                // fixed so far, find the bin of the rem-th largest, until a bin is taken whole.
                unsigned long long prefix = static_cast<unsigned long long>(bb);
                int need = rem;
                for (int shk = 32;; shk -= 8) {
                    D.t_all = shk;
                    __syncwarp();
                    if (lane == 0) {
                        ctrl->acc[b] = 0ull;
                        ctrl->T[b] = prefix;
                        ctrl->dec[b] = D;
                        mbar_arrive(shk == 32 ? &ctrl->cdec[b] : &ctrl->cdec2[b]);
                    }
                    stream_wait(ctrl, &ctrl->hand[b], (hand_par >> b) & 1u);
                    const int4 h0 = reinterpret_cast<const int4 *>(hist)[2 * grp];
                    const int4 h1 = reinterpret_cast<const int4 *>(hist)[2 * grp + 1];
                    const int c[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
                    int b2 = 0, c2 = 0, r2 = 0;
                    stream_boundary(c, lane, need, b2, c2, r2);
                    reinterpret_cast<int4 *>(hist)[2 * grp] = make_int4(0, 0, 0, 0);
                    reinterpret_cast<int4 *>(hist)[2 * grp + 1] = make_int4(0, 0, 0, 0);
                    prefix = (prefix << 8) | static_cast<unsigned long long>(b2);
                    need = r2;
                    if (c2 == r2 || shk == 0) {   // the whole bin is taken (keys are distinct: at the last digit at the latest)
                        D.kind = 2;
                        __syncwarp();
                        if (lane == 0) {
                            ctrl->T[b] = prefix << shk;
                            ctrl->dec[b] = D;
                            mbar_arrive(&ctrl->cdec2[b]);
                        }
                        hand_par ^= 1u << b;
                        break;
                    }
                    hand_par ^= 1u << b;
                }
            }
            p_listing = listing;
            p_rem = rem;
            p_sgn = D.sgn_c;
            p_m = fin.z;
            p_layer = fin.y;
            p_ec = ec - static_cast<long long>(D.sgn_c) * k_eff * kOne;
            p_s = s;
        }
        bool bulk_prev = false;
        if (f_valid) {
            // ---- channel i - 1: exact rank inside the boundary bin, then the codes leave
            const int pb = b ^ 1, pj = (i + 3) & 3;
            const LayerDesc &L = tbl.layers[f_layer];
            unsigned char *codes = smem + lay.off_codes + static_cast<size_t>(pj) * lay.c_bytes;
            float *kerr = L.kerr ? L.kerr + static_cast<size_t>(f_m) * L.N : nullptr;
            {   // the threads that said they are concerned: their flips, their members of the boundary bin
                const int qn = min(ctrl->qcount[pb], kStreamQueueCap);
                if (qn > 0) {
                    const StreamDecision Dp = ctrl->dec[pb];
                    const unsigned long long Tp = ctrl->T[pb];
                    const unsigned char *hset = held_scratch + static_cast<size_t>(blockIdx.x) * (kStreamHeldSets * kStreamHeldBytes) + pj * kStreamHeldBytes;
                    StreamListEntry *bl = reinterpret_cast<StreamListEntry *>(smem + lay.off_list) + pb * kStreamListCap;
                    for (int x = lane; x < qn; x += 32)
                        stream_flip_thread(ctrl->queue[pb][x], Dp, Tp, hset, codes, kerr, bl, &ctrl->lcount[pb]);
                }
                __syncwarp();
                if (lane == 0) ctrl->qcount[pb] = 0;
            }
            if (f_listing) {   // the first `f_rem` of the bin's members are flipped
                const StreamListEntry *blist = reinterpret_cast<const StreamListEntry *>(smem + lay.off_list) + pb * kStreamListCap;
                const int cnt = min(ctrl->lcount[pb], kStreamListCap);
                for (int x = lane; x < cnt; x += 32) {
                    const StreamListEntry me = blist[x];
                    int rank = 0;
                    for (int y = 0; y < cnt; ++y) {
                        const StreamListEntry o = blist[y];
                        rank += (o.a > me.a || (o.a == me.a && o.n < me.n)) ? 1 : 0;
                    }
                    if (rank < f_rem) {
                        SQ_DBG(me.pos >= 0 && me.pos < L.NK && me.n >= 0 && me.n < L.N, 23);   // a listed candidate of this channel
                        unsigned char *bp = codes + min(max(me.pos, 0), lay.c_bytes - 1);
                        *bp = static_cast<unsigned char>(*bp - f_sgn);
                        if (kerr) kerr[me.n] = __fmul_rn(__int2float_rn(me.e - f_sgn * kOne), 0x1p-30f);
                    }
                }
                __syncwarp();
                if (lane == 0) ctrl->lcount[pb] = 0;
            }
            unsigned char *cg = reinterpret_cast<unsigned char *>(L.codes) + static_cast<size_t>(f_m) * L.NK;
            // a row that is not a whole number of 16-byte words, or does not start on one, leaves by plain stores
            bulk_prev = (reinterpret_cast<uintptr_t>(cg) & 15) == 0 && (L.NK & 15) == 0;
            if (!bulk_prev) {
                if ((reinterpret_cast<uintptr_t>(cg) & 3) == 0) {   // N is a multiple of four: so is the row
                    for (int q = lane; q < (L.NK >> 2); q += 32)
                        reinterpret_cast<unsigned *>(cg)[q] = reinterpret_cast<const unsigned *>(codes)[q];
                } else {
                    for (int q = lane; q < L.NK; q += 32) cg[q] = codes[q];
                }
            }
            __syncwarp();
            if (lane == 0) {
                if (bulk_prev) bulk_store(cg, codes, static_cast<unsigned>(L.NK));
                L.scales[f_m] = f_s;
                if (L.cerr) L.cerr[f_m] = __fmul_rn(__ll2float_rn(f_ec), 0x1p-30f);
            }
        }
        // The codes buffer of channel i - 1 is free once the bulk copy has read it.  Nobody waits for that by
        // name: the buffer's next writers (step i + 3) have by then waited for the decision of channel i + 1,
        // which goes out after this point.
        if (f_valid && bulk_prev && lane == 0) bulk_store_wait();
        __syncwarp();
        p_valid = item >= 0;
        if (item < 0) break;
    }
}

}  // namespace sq
