// Device code of the SQuant solver for sm_100a.
//
// One cooperative thread group (a warp, or 64..512 threads joined by a named barrier) owns one
// output channel: it stages the channel's N*K weights in shared memory while taking their
// absmax, then every thread quantizes whole kernels (SQuant-E, SQuant-K and the candidate of
// Algorithm 3 are thread-local), and the group finishes with the channel step (SQuant-C): an
// exact integer sum and a radix select over the kernels' candidate keys.
//
// All decisions after the fp32 division are integer arithmetic on perturbations in units of
// 2^-30, so the result does not depend on how the work is split over threads.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace sq {

constexpr int kCtaThreads = 512;
constexpr int kOne = 1 << 30;   // perturbation 1.0 in fixed point
constexpr int kHalf = 1 << 29;  // perturbation 0.5
constexpr int kHistBins = 256;
constexpr int kIdxBits = 18;    // a channel has fewer than 2^18 kernels (host checks N*K < 2^16)
constexpr unsigned kFull = 0xffffffffu;

// One layer as the kernel sees it.  Offsets are bytes inside a group's shared-memory slice.
struct LayerDesc {
    const float *w;
    int8_t *codes;
    float *scales;
    float *kerr;
    float *cerr;
    int32_t M, N, K, NK;
    int32_t g;            // threads per channel group: 32, 64, 128, 256 or 512
    int32_t g_shift;      // log2(g)
    int32_t slice_bytes;  // shared memory per group
    int32_t off_codes, off_ev, off_vv, off_vi, off_hist, off_red;
};

// One CTA: channels ch0 .. ch0 + 512/g - 1 of one layer, one per group.
struct Item {
    int32_t layer;
    int32_t ch0;
};

struct Group {
    int g;    // threads in the group
    int t;    // this thread's index inside the group
    int bar;  // named barrier of the group (groups wider than a warp)
    __device__ __forceinline__ void sync() const
    {
        if (g == 32) __syncwarp();
        else asm volatile("bar.sync %0, %1;" ::"r"(bar), "r"(g) : "memory");
    }
};

// ---------------------------------------------------------------- group-wide reductions
// `red` points at 16 eight-byte slots owned by the group.
__device__ __forceinline__ float group_absmax(const Group &G, float v, void *red)
{
    unsigned u = __reduce_max_sync(kFull, __float_as_uint(v));  // v >= 0: uint order = float order
    if (G.g > 32) {
        unsigned *r = reinterpret_cast<unsigned *>(red);
        if ((G.t & 31) == 0) r[G.t >> 5] = u;
        G.sync();
        const int nw = G.g >> 5;
        u = 0;
        for (int i = 0; i < nw; ++i) u = max(u, r[i]);
        G.sync();
    } else {
        __syncwarp();
    }
    return __uint_as_float(u);
}

__device__ __forceinline__ long long group_sum(const Group &G, long long v, void *red)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    if (G.g > 32) {
        long long *r = reinterpret_cast<long long *>(red);
        if ((G.t & 31) == 0) r[G.t >> 5] = v;
        G.sync();
        const int nw = G.g >> 5;
        v = 0;
        for (int i = 0; i < nw; ++i) v += r[i];
        G.sync();
    }
    return v;
}

// ---------------------------------------------------------------- SQuant-E on one element
// Algorithm 1 "Scale and SQuant-E": x = w / s (IEEE division), code = round-half-even(x),
// perturbation = code - x, converted once to units of 2^-30.  With s = absmax / qmax,
// |x| < qmax + 0.5 always holds, so the clip of Sec. 2.2 never changes the code.
__device__ __forceinline__ void squant_e(float w, float s, int &q, int &P)
{
    const float x = __fdiv_rn(w, s);
    const float qf = rintf(x);
    const float p = __fsub_rn(qf, x);                    // exact: qf is a neighbour integer of x
    q = __float2int_rn(qf);
    P = __float2int_rn(__fmul_rn(p, 1073741824.0f));     // scaling by 2^30 is exact
}

// k = round(|e|) of Algorithm 2 with "exactly one half" going to the smaller count.
__device__ __forceinline__ int flip_count(long long abs_e)
{
    return static_cast<int>((abs_e + (kHalf - 1)) >> 30);
}

// ---------------------------------------------------------------- one kernel, any K (in smem)
// SQuant-K (Algorithm 2) and the candidate of Algorithm 3 for the kernel whose K weights sit at
// wk.  The weights are overwritten by their integer perturbations; codes go to ck.
// A flipped element changes the sign of its perturbation, so it leaves the candidate set by
// itself and "largest remaining same-sign perturbation, lowest index first" is the next one in
// Algorithm 2's top-k order.
__device__ __forceinline__ void kernel_generic(float *wk, int K, float s, bool do_k, int8_t *ck,
                                               long long &e_out, int &v_out, int &idx_out)
{
    int *Pk = reinterpret_cast<int *>(wk);
    long long e = 0;
    for (int i = 0; i < K; ++i) {
        int q, P;
        squant_e(wk[i], s, q, P);
        ck[i] = static_cast<int8_t>(q);
        Pk[i] = P;
        e += P;
    }
    int v = 0, idx = 0;
    if (e != 0) {
        const int sgn = e > 0 ? 1 : -1;
        const long long abs_e = e > 0 ? e : -e;
        const int k = do_k ? flip_count(abs_e) : 0;
        int flips = 0, last = -1, cand = -1;
        for (int r = 0; r <= k; ++r) {
            int best = 0, bi = -1;
            for (int i = 0; i < K; ++i) {
                const int key = sgn * Pk[i];
                if (key > best) { best = key; bi = i; }
            }
            if (bi < 0) break;
            if (r < k) {
                Pk[bi] -= sgn * kOne;
                ck[bi] = static_cast<int8_t>(ck[bi] - sgn);
                last = bi;
                ++flips;
            } else {
                cand = bi;
            }
        }
        e -= static_cast<long long>(sgn) * flips * kOne;
        if (static_cast<long long>(flips) * kOne > abs_e) {   // Over SQuant: flip back candidate
            idx = last;
            v = Pk[last];
        } else if (cand >= 0) {                               // Under SQuant: next un-flipped
            idx = cand;
            v = Pk[cand];
        }
    }
    e_out = e;
    v_out = v;
    idx_out = idx;
}

// ---------------------------------------------------------------- one kernel, K in registers
template <int K>
__device__ __forceinline__ void kernel_regs(const float *wk, float s, bool do_k, int8_t *ck,
                                            long long &e_out, int &v_out, int &idx_out)
{
    int P[K], q[K];
    long long e = 0;
#pragma unroll
    for (int i = 0; i < K; ++i) {
        squant_e(wk[i], s, q[i], P[i]);
        e += P[i];
    }
    int v = 0, idx = 0;
    if (e != 0) {
        const int sgn = e > 0 ? 1 : -1;
        const long long abs_e = e > 0 ? e : -e;
        const int k = do_k ? flip_count(abs_e) : 0;
        int flips = 0, last = -1, cand = -1;
        for (int r = 0; r <= k; ++r) {
            int best = 0, bi = -1;
#pragma unroll
            for (int i = 0; i < K; ++i) {
                const int key = sgn * P[i];
                if (key > best) { best = key; bi = i; }
            }
            if (bi < 0) break;
            if (r < k) {
#pragma unroll
                for (int i = 0; i < K; ++i)
                    if (i == bi) { P[i] -= sgn * kOne; q[i] -= sgn; }
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
#pragma unroll
            for (int i = 0; i < K; ++i)
                if (i == pick) v = P[i];
        }
    }
#pragma unroll
    for (int i = 0; i < K; ++i) ck[i] = static_cast<int8_t>(q[i]);
    e_out = e;
    v_out = v;
    idx_out = idx;
}

// ---------------------------------------------------------------- SQuant-C selection
// Key of a kernel's candidate in Algorithm 2's order on the channel: larger |v| first, equal |v|
// by lower kernel index.  0 = not a candidate for this sign.
__device__ __forceinline__ unsigned long long cand_key(int v, int sgn_c, int n)
{
    const int a = v * sgn_c;   // > 0 iff v has the sign of the channel sum
    if (a <= 0) return 0ull;
    return (static_cast<unsigned long long>(static_cast<unsigned>(a)) << kIdxBits) |
           static_cast<unsigned long long>(((1 << kIdxBits) - 1) - n);
}

// Histogram bins are stored swizzled so that the scanning warp (lane l sums 8 consecutive bins)
// reads without bank conflicts.
__device__ __forceinline__ int hist_slot(int bin) { return ((bin & 7) << 5) | (bin >> 3); }

// Finds the threshold T such that exactly min(kc, #candidates) candidate keys are >= T (keys are
// distinct).  Most-significant-digit radix select, 8 bits per pass over the 48-bit keys, leaving
// early once the boundary bin is taken whole.  Returns the number of kernels to flip (0: none).
// All threads of the group must call it; vv holds the candidates of kernels 0..N-1.
__device__ __forceinline__ int select_threshold(const Group &G, const int *vv, int N, int sgn_c,
                                                int kc, int *hist, int *bc,
                                                unsigned long long &T_out)
{
    unsigned long long prefix = 0;   // digits already fixed (bits above the current digit)
    int need = kc, k_eff = 0;
    T_out = ~0ull;
    for (int pass = 0; pass < 6; ++pass) {
        const int sh = 40 - 8 * pass;
        for (int i = G.t; i < kHistBins; i += G.g) hist[i] = 0;
        G.sync();
        for (int n = G.t; n < N; n += G.g) {
            const unsigned long long ck = cand_key(vv[n], sgn_c, n);
            if (ck != 0 && (pass == 0 || (ck >> (sh + 8)) == prefix))
                atomicAdd(&hist[hist_slot(static_cast<int>(ck >> sh) & 255)], 1);
        }
        G.sync();
        if (G.t < 32) {
            const int lane = G.t;
            const int grp = 31 - lane;   // lane 0 owns the highest 8 bins
            int c[8], s8 = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { c[j] = hist[(j << 5) | grp]; s8 += c[j]; }
            int incl = s8;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(kFull, incl, o);
                if (lane >= o) incl += t;
            }
            const int total = __shfl_sync(kFull, incl, 31);
            const int want = pass == 0 ? min(kc, total) : need;
            const unsigned bal = __ballot_sync(kFull, incl >= want);
            if (want <= 0) {
                if (lane == 0) { bc[0] = -1; bc[1] = 0; bc[2] = 0; bc[3] = 0; }
            } else {
                const int sel = __ffs(bal) - 1;
                if (lane == sel) {
                    int cum = incl - s8, b = -1, cb = 0;
#pragma unroll
                    for (int j = 7; j >= 0; --j) {
                        if (b < 0) {
                            if (cum + c[j] >= want) { b = grp * 8 + j; cb = c[j]; }
                            else cum += c[j];
                        }
                    }
                    bc[0] = b;            // boundary bin
                    bc[1] = want - cum;   // keys still to take inside it
                    bc[2] = cb;           // keys in it
                    bc[3] = want;
                }
            }
        }
        G.sync();
        const int b = bc[0], rem = bc[1], cb = bc[2];
        if (pass == 0) k_eff = bc[3];
        if (b < 0) return 0;
        prefix = (prefix << 8) | static_cast<unsigned long long>(b);
        need = rem;
        if (cb == rem) {   // the whole boundary bin is taken
            T_out = prefix << sh;
            break;
        }
    }
    return k_eff;
}

// ---------------------------------------------------------------- one output channel
template <int KT>
__device__ __forceinline__ void quantize_channel(const LayerDesc &L, int m, const Group &G,
                                                 unsigned char *slice, int qmax, unsigned mode)
{
    const int K = KT ? KT : L.K;
    const int N = L.N, NK = L.NK;
    float *wbuf = reinterpret_cast<float *>(slice);
    int8_t *cbuf = reinterpret_cast<int8_t *>(slice + L.off_codes);
    int *ev = reinterpret_cast<int *>(slice + L.off_ev);
    int *vv = reinterpret_cast<int *>(slice + L.off_vv);
    unsigned short *vi = reinterpret_cast<unsigned short *>(slice + L.off_vi);
    int *hist = reinterpret_cast<int *>(slice + L.off_hist);
    unsigned char *red = slice + L.off_red;
    int *bc = reinterpret_cast<int *>(red + 128);

    // ---- stage the channel in shared memory, absmax on the way
    const float *wg = L.w + static_cast<size_t>(m) * NK;
    float amax = 0.0f;
    if ((reinterpret_cast<uintptr_t>(wg) & 15) == 0) {
        const int nv = NK >> 2;
        const float4 *src = reinterpret_cast<const float4 *>(wg);
        float4 *dst = reinterpret_cast<float4 *>(wbuf);
        for (int i = G.t; i < nv; i += G.g) {
            const float4 t = __ldcs(src + i);
            dst[i] = t;
            amax = fmaxf(fmaxf(amax, fabsf(t.x)), fmaxf(fabsf(t.y), fmaxf(fabsf(t.z), fabsf(t.w))));
        }
        for (int i = (nv << 2) + G.t; i < NK; i += G.g) {
            const float t = __ldcs(wg + i);
            wbuf[i] = t;
            amax = fmaxf(amax, fabsf(t));
        }
    } else {
        for (int i = G.t; i < NK; i += G.g) {
            const float t = __ldcs(wg + i);
            wbuf[i] = t;
            amax = fmaxf(amax, fabsf(t));
        }
    }
    amax = group_absmax(G, amax, red);   // also makes wbuf visible to the whole group
    const float s = (amax < 0x1p-100f) ? 1.0f : __fdiv_rn(amax, static_cast<float>(qmax));

    // ---- SQuant-E, SQuant-K, candidate: one thread per kernel
    // Without SQuant-K a kernel sum can reach K/2 and no longer fits 32 bits; it is then
    // emitted right here (no channel step follows: E|C is only accepted for 1x1 kernels).
    const bool do_k = (mode & 2u) != 0;
    const bool keep = do_k || KT == 1 || K == 1;
    float *kerr = L.kerr ? L.kerr + static_cast<size_t>(m) * N : nullptr;
    long long esum = 0;
    for (int n = G.t; n < N; n += G.g) {
        long long e1;
        if (KT == 1) {
            int q, P;
            squant_e(wbuf[n], s, q, P);
            cbuf[n] = static_cast<int8_t>(q);
            e1 = P;                  // a 1x1 kernel is its own candidate; ev and vv alias wbuf
            ev[n] = P;
        } else {
            int v, idx;
            if (KT == 0) kernel_generic(wbuf + static_cast<size_t>(n) * K, K, s, do_k, cbuf + static_cast<size_t>(n) * K, e1, v, idx);
            else kernel_regs<(KT > 1 ? KT : 2)>(wbuf + n * K, s, do_k, cbuf + n * K, e1, v, idx);
            if (keep) {
                ev[n] = static_cast<int>(e1);
                vv[n] = v;
                vi[n] = static_cast<unsigned short>(idx);
            } else if (kerr) {
                kerr[n] = __fmul_rn(__ll2float_rn(e1), 0x1p-30f);
            }
        }
        esum += e1;
    }

    // ---- SQuant-C: Algorithm 2 on the channel, keys = the kernels' candidates
    long long ec = 0;
    int sgn_c = 0, k_eff = 0;
    unsigned long long T = ~0ull;
    if ((mode & 4u) || L.cerr) ec = group_sum(G, esum, red);   // sync: ev / vv / cbuf visible
    else G.sync();
    if ((mode & 4u) && ec != 0) {
        sgn_c = ec > 0 ? 1 : -1;
        const long long abs_e = ec > 0 ? ec : -ec;
        const int kc = flip_count(abs_e);
        if (kc > 0) k_eff = select_threshold(G, vv, N, sgn_c, kc, hist, bc, T);
        ec -= static_cast<long long>(sgn_c) * k_eff * kOne;
    }

    // ---- apply the channel flips, emit the kernels' error sums
    if (keep && (k_eff > 0 || kerr)) {
        for (int n = G.t; n < N; n += G.g) {
            int e1 = ev[n];
            if (k_eff > 0) {
                const unsigned long long ck = cand_key(vv[n], sgn_c, n);
                if (ck != 0 && ck >= T) {
                    e1 -= sgn_c * kOne;
                    const size_t j = (KT == 1) ? n : static_cast<size_t>(n) * K + vi[n];
                    cbuf[j] = static_cast<int8_t>(cbuf[j] - sgn_c);
                }
            }
            if (kerr) kerr[n] = __fmul_rn(__int2float_rn(e1), 0x1p-30f);
        }
    }
    G.sync();

    // ---- codes, scale, channel error
    int8_t *cg = L.codes + static_cast<size_t>(m) * NK;
    if ((reinterpret_cast<uintptr_t>(cg) & 15) == 0) {
        const int nv = NK >> 4;
        const int4 *src = reinterpret_cast<const int4 *>(cbuf);
        int4 *dst = reinterpret_cast<int4 *>(cg);
        for (int i = G.t; i < nv; i += G.g) __stcs(dst + i, src[i]);
        for (int i = (nv << 4) + G.t; i < NK; i += G.g) cg[i] = cbuf[i];
    } else {
        for (int i = G.t; i < NK; i += G.g) cg[i] = cbuf[i];
    }
    if (G.t == 0) {
        L.scales[m] = s;
        if (L.cerr) L.cerr[m] = __fmul_rn(__ll2float_rn(ec), 0x1p-30f);
    }
}

// ---------------------------------------------------------------- grouped launch
__global__ void __launch_bounds__(kCtaThreads)
squant_model_kernel(const LayerDesc *__restrict__ layers, const Item *__restrict__ items, int qmax,
                    unsigned mode)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const Item it = items[blockIdx.x];
    const LayerDesc L = layers[it.layer];
    Group G;
    G.g = L.g;
    G.t = threadIdx.x & (L.g - 1);
    const int gi = threadIdx.x >> L.g_shift;
    G.bar = 1 + gi;
    const int m = it.ch0 + gi;
    if (m >= L.M) return;   // the whole group leaves together; it shares no barrier with others
    unsigned char *slice = smem + static_cast<size_t>(gi) * L.slice_bytes;
    if (L.K == 1) quantize_channel<1>(L, m, G, slice, qmax, mode);
    else if (L.K == 9) quantize_channel<9>(L, m, G, slice, qmax, mode);
    else quantize_channel<0>(L, m, G, slice, qmax, mode);
}

}  // namespace sq
