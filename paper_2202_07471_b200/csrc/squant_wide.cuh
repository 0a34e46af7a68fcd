// Cluster kernel for output channels too wide for one CTA (beyond ~37 K weights for 3x3, ~45 K
// for 1x1): a thread-block cluster of 2, 4 or 8 CTAs owns one output channel, each CTA a
// contiguous run of its kernels, staged in that CTA's shared memory.  What the channel needs as a
// whole travels through distributed shared memory (plain loads from the other CTAs' shared
// memory; no multicast anywhere): the absmax for the scale, the channel's error sum, and the
// histograms of the radix select of SQuant-C, which every CTA adds up for itself, so that all CTAs
// take the same decisions without a leader.
//
// Channels this wide can hold 2^16 and more kernels, the size from which the one element that sits
// on the edge of the clip range (|w/s| a shade above qmax) can make it into a top-k; so every
// candidate here is checked against the range, as in the CPU definition: an element whose flipped
// code would leave the range is no candidate.  Plain thread-per-kernel code, IEEE division.
#pragma once

#include <cooperative_groups.h>

#include "squant_device.cuh"

namespace sq {

namespace cg = cooperative_groups;

constexpr int kWideThreads = 512;
constexpr int kWideMaxCluster = 8;
constexpr int kWideExchangeBytes = 256;

// Shared memory of one CTA that owns `kpc` kernels of K weights.  1x1 kernels keep their
// perturbation where the weight was and need no per-kernel arrays.
struct WideLayout {
    int off_codes, off_ev, off_vv, off_vi, off_hist, off_merged, off_x, total;
};

__host__ __device__ inline WideLayout wide_layout(int kpc, int K)
{
    WideLayout w;
    const long long nk = static_cast<long long>(kpc) * K;
    long long off = (4 * nk + 15) & ~15ll;
    w.off_codes = static_cast<int>(off); off += (nk + 15) & ~15ll;
    if (K == 1) {
        w.off_ev = 0; w.off_vv = 0; w.off_vi = 0;
    } else {
        w.off_ev = static_cast<int>(off); off += (4ll * kpc + 15) & ~15ll;
        w.off_vv = static_cast<int>(off); off += (4ll * kpc + 15) & ~15ll;
        w.off_vi = static_cast<int>(off); off += (2ll * kpc + 15) & ~15ll;
    }
    w.off_hist = static_cast<int>(off); off += 4 * kHistBins;
    w.off_merged = static_cast<int>(off); off += 4 * kHistBins;
    w.off_x = static_cast<int>(off); off += kWideExchangeBytes;
    w.total = off > 0x7fffffffll ? 0x7fffffff : static_cast<int>(off);
    return w;
}

// What the CTAs of a cluster show each other.
struct WideExchange {
    unsigned amax;       // this CTA's absmax (bit pattern of a non-negative float)
    int pad;
    long long esum;      // this CTA's share of the channel's error sum
    int bc[4];           // scan result of a select pass (every CTA computes the same)
    long long red[kWideThreads / 32];   // block reduction
};
static_assert(sizeof(WideExchange) <= kWideExchangeBytes, "exchange block larger than its place in shared memory");

// One output channel per cluster; grid = channels * cluster size.
__global__ void __launch_bounds__(kWideThreads, 1)
squant_wide_kernel(const LayerDesc L, int qmax, unsigned mode, int kpc)
{
    extern __shared__ __align__(16) unsigned char smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const int C = static_cast<int>(cluster.num_blocks()), rank = static_cast<int>(cluster.block_rank());
    const int m = static_cast<int>(blockIdx.x) / C;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = L.K, N = L.N;
    const int n0 = min(rank * kpc, N), nloc = min(N - n0, kpc);   // this CTA's kernels: n0 .. n0 + nloc - 1
    const int eloc = nloc * K;
    const WideLayout lay = wide_layout(kpc, K);
    float *wbuf = reinterpret_cast<float *>(smem);
    int *Pbuf = reinterpret_cast<int *>(smem);
    int8_t *cbuf = reinterpret_cast<int8_t *>(smem + lay.off_codes);
    int *ev = reinterpret_cast<int *>(smem + lay.off_ev);
    int *vv = reinterpret_cast<int *>(smem + lay.off_vv);
    unsigned short *vi = reinterpret_cast<unsigned short *>(smem + lay.off_vi);
    int *hist = reinterpret_cast<int *>(smem + lay.off_hist);
    int *merged = reinterpret_cast<int *>(smem + lay.off_merged);
    WideExchange *xc = reinterpret_cast<WideExchange *>(smem + lay.off_x);
    const int qmin = (mode & kModeWideRange) ? -qmax - 1 : -qmax;
    const bool do_k = (mode & 2u) != 0;

    // ---- stage this CTA's run of the channel, take its absmax
    const float *wg = L.w + static_cast<size_t>(m) * L.NK + static_cast<size_t>(n0) * K;
    float amax = 0.0f;
    for (int i = tid; i < eloc; i += kWideThreads) {
        const float t = __ldcs(wg + i);
        wbuf[i] = t;
        amax = fmaxf(amax, fabsf(t));
    }
    if (tid == 0) xc->amax = 0u;
    __syncthreads();
    {
        const unsigned wmax = __reduce_max_sync(kFull, __float_as_uint(amax));
        if (lane == 0) atomicMax(&xc->amax, wmax);
    }
    __syncthreads();
    cluster.sync();   // every CTA's absmax is in place
    float s;
    if (L.sin) {      // Algorithm 1 with its scale as an input
        s = L.sin[m];
        if (!(s > 0.0f && s < __int_as_float(0x7f800000))) s = 1.0f;
    } else {
        unsigned a = 0u;
        for (int c = 0; c < C; ++c) a = max(a, cluster.map_shared_rank(xc, c)->amax);
        const float am = __uint_as_float(a);
        s = (am < 0x1p-100f) ? 1.0f : __fdiv_rn(am, static_cast<float>(qmax));
    }

    // ---- SQuant-E, SQuant-K, candidates: one thread per kernel
    float *kerr = L.kerr ? L.kerr + static_cast<size_t>(m) * N + n0 : nullptr;
    long long esum = 0;
    for (int n = tid; n < nloc; n += kWideThreads) {
        long long e;
        int v, idx;
        kernel_clip(wbuf + static_cast<size_t>(n) * K, K, s, do_k, qmin, qmax, cbuf + static_cast<size_t>(n) * K, e, v, idx);
        if (K > 1) {   // a kernel that SQuant-C can flip has a candidate, hence |e'| <= 1/2: its 32-bit copy is exact
            ev[n] = static_cast<int>(max(min(e, 0x7fffffffll), -0x7fffffffll));
            vv[n] = v;
            vi[n] = static_cast<unsigned short>(idx);
        }
        if (kerr) kerr[n] = __fmul_rn(__ll2float_rn(e), 0x1p-30f);
        esum += e;
    }
    // channel sum: block reduction, then over the cluster
    for (int o = 16; o > 0; o >>= 1) esum += __shfl_xor_sync(kFull, esum, o);
    if (lane == 0) xc->red[warp] = esum;
    __syncthreads();
    if (tid == 0) {
        long long t = 0;
        for (int i = 0; i < kWideThreads / 32; ++i) t += xc->red[i];
        xc->esum = t;
    }
    __syncthreads();
    cluster.sync();
    long long ec = 0;
    for (int c = 0; c < C; ++c) ec += cluster.map_shared_rank(xc, c)->esum;

    // Key of kernel n (local index) in Algorithm 2's order on the channel for direction sgn_c, 0
    // if it is no candidate.  For 1x1 kernels the element is its own candidate and the range
    // check is made here; larger kernels checked their candidate when they chose it (flipping an
    // Over-SQuant candidate back, or an Under-SQuant one on, keeps the code in range).
    auto key_of = [&](int n, int sgn_c) -> unsigned long long {
        if (K == 1) {
            const int fl = cbuf[n] - sgn_c;
            if (fl < qmin || fl > qmax) return 0ull;
            return cand_key(Pbuf[n], sgn_c, n0 + n);
        }
        return cand_key(vv[n], sgn_c, n0 + n);
    };

    // ---- SQuant-C: radix select over the candidates of the whole channel
    int sgn_c = 0, k_eff = 0;
    unsigned long long T = ~0ull;
    if ((mode & 4u) && ec != 0) {
        sgn_c = ec > 0 ? 1 : -1;
        const long long abs_e = ec > 0 ? ec : -ec;
        const int kc = static_cast<int>(min((abs_e + (kHalf - 1)) >> 30, 1ll << 30));
        if (kc > 0) {
            unsigned long long prefix = 0;
            int need = kc;
            for (int pass = 0; pass < 6; ++pass) {
                const int sh = 40 - 8 * pass;
                for (int i = tid; i < kHistBins; i += kWideThreads) hist[i] = 0;
                __syncthreads();
                for (int n = tid; n < nloc; n += kWideThreads) {
                    const unsigned long long ck = key_of(n, sgn_c);
                    if (ck != 0 && (pass == 0 || (ck >> (sh + 8)) == prefix))
                        atomicAdd(&hist[hist_slot(static_cast<int>(ck >> sh) & 255)], 1);
                }
                __syncthreads();
                cluster.sync();   // every CTA's histogram of this pass is complete
                for (int i = tid; i < kHistBins; i += kWideThreads) {
                    int t = 0;
                    for (int c = 0; c < C; ++c) t += cluster.map_shared_rank(hist, c)[i];
                    merged[i] = t;
                }
                __syncthreads();
                if (tid < 32) {   // scan, highest bins first: lane 0 owns the highest 8 bins
                    const int grp = 31 - lane;
                    int c8[8], s8 = 0;
#pragma unroll
                    for (int j = 0; j < 8; ++j) { c8[j] = merged[(j << 5) | grp]; s8 += c8[j]; }
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
                        if (lane == 0) { xc->bc[0] = -1; xc->bc[1] = 0; xc->bc[2] = 0; xc->bc[3] = 0; }
                    } else if (lane == __ffs(bal) - 1) {
                        int cum = incl - s8, b = -1, cb = 0;
#pragma unroll
                        for (int j = 7; j >= 0; --j) {
                            if (b < 0) {
                                if (cum + c8[j] >= want) { b = grp * 8 + j; cb = c8[j]; }
                                else cum += c8[j];
                            }
                        }
                        xc->bc[0] = b; xc->bc[1] = want - cum; xc->bc[2] = cb; xc->bc[3] = want;
                    }
                }
                __syncthreads();
                const int b = xc->bc[0], rem = xc->bc[1], cb = xc->bc[2];
                if (pass == 0) k_eff = xc->bc[3];
                cluster.sync();   // all CTAs have read the histograms: they may be cleared for the next pass
                if (b < 0) { k_eff = 0; break; }
                prefix = (prefix << 8) | static_cast<unsigned long long>(b);
                need = rem;
                if (cb == rem) {   // the whole boundary bin is taken
                    T = prefix << sh;
                    break;
                }
            }
            ec -= static_cast<long long>(sgn_c) * k_eff * kOne;
        }
    }

    // ---- apply the channel flips to this CTA's kernels
    if (k_eff > 0) {
        for (int n = tid; n < nloc; n += kWideThreads) {
            const unsigned long long ck = key_of(n, sgn_c);
            if (ck != 0 && ck >= T) {
                const size_t j = K == 1 ? static_cast<size_t>(n) : static_cast<size_t>(n) * K + vi[n];
                cbuf[j] = static_cast<int8_t>(cbuf[j] - sgn_c);
                const int e1 = (K == 1 ? Pbuf[n] : ev[n]) - sgn_c * kOne;
                if (kerr) kerr[n] = __fmul_rn(__int2float_rn(e1), 0x1p-30f);
            }
        }
    }
    __syncthreads();

    // ---- emit this CTA's run of the channel
    const size_t e0 = static_cast<size_t>(n0) * K;   // first element of the run inside the channel (even: kpc * K is)
    if (L.deq) {
        float *dg = L.deq + static_cast<size_t>(m) * L.NK + e0;
        for (int i = tid; i < eloc; i += kWideThreads) dg[i] = __fmul_rn(__int2float_rn(cbuf[i]), s);
    }
    if (L.deq16) {
        uint16_t *dg = L.deq16 + static_cast<size_t>(m) * L.NK + e0;
        for (int i = tid; i < eloc; i += kWideThreads) dg[i] = static_cast<uint16_t>(bf16_bits(__fmul_rn(__int2float_rn(cbuf[i]), s)));
    }
    if (mode & kModePackInt4) {   // two codes per byte, low nibble = even flat index
        unsigned char *cg = reinterpret_cast<unsigned char *>(L.codes) + static_cast<size_t>(m) * ((L.NK + 1) >> 1) + (e0 >> 1);
        const int pairs = eloc >> 1;
        for (int i = tid; i < pairs; i += kWideThreads)
            cg[i] = static_cast<unsigned char>((cbuf[2 * i] & 15) | (cbuf[2 * i + 1] << 4));
        if ((eloc & 1) && tid == 0) cg[pairs] = static_cast<unsigned char>(cbuf[eloc - 1] & 15);   // only the channel's last run can be odd
    } else {
        int8_t *cg = L.codes + static_cast<size_t>(m) * L.NK + e0;
        if (((reinterpret_cast<uintptr_t>(cg) | reinterpret_cast<uintptr_t>(cbuf)) & 15) == 0) {
            const int nv = eloc >> 4;
            for (int i = tid; i < nv; i += kWideThreads) __stcs(reinterpret_cast<int4 *>(cg) + i, reinterpret_cast<const int4 *>(cbuf)[i]);
            for (int i = (nv << 4) + tid; i < eloc; i += kWideThreads) cg[i] = cbuf[i];
        } else {
            for (int i = tid; i < eloc; i += kWideThreads) cg[i] = cbuf[i];
        }
    }
    if (rank == 0 && tid == 0) {
        L.scales[m] = s;
        if (L.cerr) L.cerr[m] = __fmul_rn(__ll2float_rn(ec), 0x1p-30f);
    }
    cluster.sync();   // no CTA leaves while another may still read its shared memory
}

}  // namespace sq
