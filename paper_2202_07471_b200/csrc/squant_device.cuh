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

constexpr int kCtaThreads = 256;   // four CTAs per SM (64 registers): measured best for whole models against 512 x 2 and 128 x 8
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
    float *deq;
    const float *sin;     // caller-supplied scales, or null: absmax scales
    uint16_t *deq16;      // bfloat16 code * s, or null
    int32_t M, N, K, NK;
    int32_t g;            // threads per channel group: 32, 64, 128 or 256
    int32_t g_shift;      // log2(g)
    int32_t slice_bytes;  // shared memory per group
    int32_t off_codes, off_ev, off_vv, off_vi, off_hist, off_red;
};

// One CTA: channels ch0 .. ch0 + 256/g - 1 of one layer, one per group.
struct Item {
    int32_t layer;
    int32_t ch0;
};

// Everything a grouped launch needs, passed BY VALUE as a kernel parameter: the descriptors sit
// in the constant bank, so a CTA finds its work without a single global load (and nothing has
// to be allocated or uploaded).  Work items of layer l are the CTAs first_item[l] ..
// first_item[l+1]-1; item i of a layer handles channels i * (256 / g) ... of it.
constexpr int kMaxParamLayers = 96;
struct LaunchTable {
    int n_layers;
    int top_step;   // largest power of two below n_layers (0 for one layer): first step of the layer search
    int first_item[kMaxParamLayers + 1];
    LayerDesc layers[kMaxParamLayers];
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

// ---------------------------------------------------------------- checked build
// Built with -DSQUANT_DEBUG_BOUNDS (a second library, for tests on small cases), the kernels check
// the indices they form into shared memory and into the launch table against their bounds, and
// recompute every channel's error sum from its final codes and staged weights; a failed check is
// counted and its site recorded, the access it guards is skipped where it can be.  The regular
// build compiles the checks away.
__device__ unsigned g_debug_violations = 0;
__device__ int g_debug_site = 0;
#ifdef SQUANT_DEBUG_BOUNDS
__device__ __noinline__ void sq_debug_fail(int site)
{
    atomicAdd(&g_debug_violations, 1u);
    atomicCAS(&g_debug_site, 0, site);
}
#define SQ_DBG(cond, site) do { if (!(cond)) sq_debug_fail(site); } while (0)
#define SQ_DBG_OK(cond, site) ((cond) ? true : (sq_debug_fail(site), false))
#else
#define SQ_DBG(cond, site) ((void)0)
#define SQ_DBG_OK(cond, site) (true)
#endif

__device__ __forceinline__ unsigned dynamic_smem_bytes()
{
    unsigned v;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(v));
    return v;
}

// ---------------------------------------------------------------- bulk async copies (TMA)
// Set to a non-zero code by a kernel whose bounded wait on a bulk copy ran out; read and cleared
// by squant_device_status().
__device__ int g_device_status = 0;
constexpr int kWaitIters = 1 << 22;   // each try_wait itself blocks for a hardware time slice

__device__ __forceinline__ unsigned smem_addr(const void *p)
{
    return static_cast<unsigned>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(void *bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the initialised barrier is visible to the async proxy
}

// One-dimensional bulk copy global -> shared of `bytes` (multiple of 16, both sides 16-byte
// aligned, no multicast), completion counted on `bar`.
__device__ __forceinline__ void bulk_load(void *dst, const void *src, unsigned bytes, void *bar)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_addr(dst)),
                 "l"(src), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

// One arrival on `bar` (release semantics: the thread's earlier writes are visible to a thread
// that observes the phase completing).
__device__ __forceinline__ void mbar_arrive(void *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// Bounded wait for phase `parity` of `bar`.  False if the limit ran out.
__device__ __forceinline__ bool mbar_wait(void *bar, unsigned parity, int max_polls = kWaitIters)
{
    const unsigned a = smem_addr(bar);
    for (int it = 0; it < max_polls; ++it) {
        unsigned done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(a), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}

// Bulk copy shared -> global of `bytes` (multiple of 16, both sides 16-byte aligned), issued by
// one thread after the writers' barrier; the caller waits with bulk_store_wait before the shared
// memory may be reused or the CTA exits.
__device__ __forceinline__ void bulk_store(void *dst, const void *src, unsigned bytes)
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_addr(src)), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

__device__ __forceinline__ void bulk_store_wait()
{
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

// ---------------------------------------------------------------- group-wide reductions
// `red` points at 16 eight-byte slots owned by the group.
__device__ __forceinline__ float group_absmax(const Group &G, float v, void *red)
{
    // `slot` (red + 216) was zeroed before the previous group barrier
    unsigned u = __reduce_max_sync(kFull, __float_as_uint(v));  // v >= 0: uint order = float order
    if (G.g > 32) {
        unsigned *slot = reinterpret_cast<unsigned *>(static_cast<unsigned char *>(red) + 216);
        if ((G.t & 31) == 0) atomicMax(slot, u);
        G.sync();
        u = *slot;
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

// ---------------------------------------------------------------- 3x3 fast path
// The division w / s is the only expensive fp32 step, and s is constant over a channel.  With
// s2 = s * 2^-30 and y = RN(1 / s2) (one IEEE reciprocal per channel), the sequence
//     X0 = RN(w * y);  r = fma(-X0, s2, w);  X = fma(r, y, X0)
// returns the correctly rounded quotient RN(w / s2) = RN(w / s) * 2^30 (Markstein's theorem: y
// is a correctly rounded reciprocal, X0 is within one ulp, r is exact).  It needs s2 and y to be
// normal numbers; the caller takes this path only for 2^-60 <= s <= 2^60.  The quotient comes
// out already scaled to the fixed-point unit, so
//     t  = X + kMagic     rounds X to a multiple of 2^30, ties to even (ulp of t is 2^30)
//     qX = t - kMagic     = code * 2^30, exactly
//     P  = cvt.rni(qX - X)   the perturbation in 2^-30 units (the difference is exact)
// and the low byte of t's bit pattern is the code in two's complement.
constexpr unsigned kRedoMark = 0xffu;   // element index stored for a kernel that awaits its exact redo
constexpr float kMagic = 0x1.8p53f;   // 1.5 * 2^53: mantissa field 0x400000, low byte 0

__device__ __forceinline__ float div_scaled(float w, float y, float s2)
{
    const float x0 = __fmul_rn(w, y);
    const float r = __fmaf_rn(-x0, s2, w);
    return __fmaf_rn(r, y, x0);
}

__device__ __forceinline__ void squant_e_fastf(float w, float y, float s2, unsigned &tbits, float &Pf)
{
    const float X = div_scaled(w, y, s2);
    const float t = __fadd_rn(X, kMagic);
    const float qX = __fsub_rn(t, kMagic);
    Pf = __fsub_rn(qX, X);   // exact; |Pf| <= 2^29 (+ one ulp of qmax * 2^30 for the absmax element)
    tbits = __float_as_uint(t);
}

__device__ __forceinline__ void squant_e_fast(float w, float y, float s2, unsigned &tbits, int &P)
{
    float Pf;
    squant_e_fastf(w, y, s2, tbits, Pf);
    P = __float2int_rn(Pf);
}

// The same on two weights at once with sm_100's packed fp32x2 arithmetic: each instruction
// yields two IEEE round-to-nearest results, identical to the scalar sequence above, for one
// issue slot.  E2 holds the channel's constants as pairs.
struct E2 {
    float2 y, ns2, magic, nmagic, neg1;
};

__device__ __forceinline__ E2 make_e2(float y, float s2)
{
    E2 c;
    c.y = make_float2(y, y);
    c.ns2 = make_float2(-s2, -s2);
    c.magic = make_float2(kMagic, kMagic);
    c.nmagic = make_float2(-kMagic, -kMagic);
    c.neg1 = make_float2(-1.0f, -1.0f);
    return c;
}

__device__ __forceinline__ void squant_e_fast2(float2 w, const E2 &c, float2 &t, float2 &Pf)
{
    const float2 x0 = __fmul2_rn(w, c.y);
    const float2 r = __ffma2_rn(x0, c.ns2, w);      // w - x0 * s2, exact
    const float2 X = __ffma2_rn(r, c.y, x0);        // RN(w / s2)
    t = __fadd2_rn(X, c.magic);
    const float2 qX = __fadd2_rn(t, c.nmagic);
    Pf = __ffma2_rn(X, c.neg1, qX);                 // qX - X, exact
}

// Exact SQuant-K + Algorithm 3 on one 3x3 kernel from its weights in shared memory; codes are
// written as bytes.  Used for the few kernels the fast selection hands back; kept out of line so
// that the common path stays small.
struct KernelOut {
    int e, v, idx;
};

// kDiv = false: SQuant-E by the reciprocal sequence (y, s2 as in squant_e_fast); kDiv = true: by
// the plain IEEE division, for scales outside the reciprocal's range (y is the scale s then).
template <bool kDiv>
__device__ __noinline__ KernelOut kernel9_exact_t(const float *wk, float y, float s2, unsigned char *cb)
{
    int P[9], q[9];
    long long e = 0;
#pragma unroll
    for (int i = 0; i < 9; ++i) {
        if (kDiv) {
            squant_e(wk[i], y, q[i], P[i]);
        } else {
            unsigned tb;
            squant_e_fast(wk[i], y, s2, tb, P[i]);
            q[i] = static_cast<int>(tb & 255u);
        }
        e += P[i];
    }
    int v = 0, idx = 0;
    if (e != 0) {
        const int sgn = e > 0 ? 1 : -1;
        const long long abs_e = e > 0 ? e : -e;
        const int k = flip_count(abs_e);
        int flips = 0, last = -1, cand = -1;
        for (int r = 0; r <= k; ++r) {
            int best = 0, bi = -1;
#pragma unroll
            for (int i = 0; i < 9; ++i) {
                const int key = sgn * P[i];
                if (key > best) { best = key; bi = i; }
            }
            if (bi < 0) break;
            if (r < k) {
#pragma unroll
                for (int i = 0; i < 9; ++i)
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
            for (int i = 0; i < 9; ++i)
                if (i == pick) v = P[i];
        }
    }
#pragma unroll
    for (int i = 0; i < 9; ++i) cb[i] = static_cast<unsigned char>(q[i]);
    KernelOut o;
    o.e = static_cast<int>(e);
    o.v = v;
    o.idx = idx;
    return o;
}

__device__ __forceinline__ KernelOut kernel9_exact(const float *wk, float y, float s2, unsigned char *cb)
{
    return kernel9_exact_t<false>(wk, y, s2, cb);
}

// Fast SQuant-K + Algorithm 3 on one 3x3 kernel whose exact perturbations Pf[0..8] (floats, in
// 2^-30 units, before the conversion to integers) are in registers and whose code bytes are
// already staged at cb.  Straight-line on purpose: every lane runs the same instructions; a
// kernel it cannot settle is reported (return value true) and redone by kernel9_exact.
//
// Sign.  A float sum of the perturbations (within 4096 units of the exact sum) gives the sign
// used to normalise the elements; the exact |e| is then the integer sum of the normalised
// elements (mod 2^32).  If the float sign was wrong (|e| <= 4096) that sum wraps to >= 2^32 -
// 4096 and the kernel is reported; |float sum| >= 3.75 * 2^30 (where 32 bits could wrap) too.
//
// Decisions, all from the exact |e|: jx = (|e| - t) >> 29 with t = (|e| is no multiple of 2^30),
// i.e. floor(|e| / 2^29) with "exactly k + 1/2" falling to the lower value.  Then the flip count
// of Algorithm 2 is k = (jx + 1) / 2, the kernel is Over SQuant iff jx is odd, and the candidate
// of Algorithm 3 is the element of rank c = (jx + 2) / 2 (the last flipped one when Over, the
// first un-flipped one otherwise).  Every jx = 0..7 is handled (k <= 4, c <= 4); what is left for
// the exact routine is |e| >= 3.75, uncertified keys and a wrong float sign: about one kernel in
// 10^5 on random weights.
//
// Selection.  Keys are the sign-normalised integer perturbations with the element index folded
// into their low four bits, (P & ~15) | (15 - i): distinct, and ordered like Algorithm 2's
// (P descending, index ascending) among elements whose low four bits are zero.  That holds for
// every element with P >= 2^27: its quotient w/s * 2^30 is an fp32 number of magnitude >= 2^27,
// hence a multiple of 16.  So if the key of rank c is >= 2^27 the first c ranks are exact, and
// so is the candidate's value (the key without its index bits); otherwise the kernel is
// reported.  The four largest keys come from a 3x3 sorting tableau: sort each triple (rows), then
// the columns; an entry in row i, column j has at least i * j - 1 entries above it, so the top
// four of nine lie in row 1, column 1 and position (2, 2) (28 operations).
__device__ __forceinline__ bool kernel9_select(const float (&Psf)[9], float ef, unsigned char *cb,
                                               int &e_out, int &v_out, unsigned &idx_out)
{
    // Psf[i] = Pf[i] * copysign(1, ef): the perturbations normalised to the sign of the float sum
    const int sgn = (__float_as_int(ef) >> 31) | 1;
    int a[9];
    unsigned eabs = 0;   // |e| mod 2^32
#pragma unroll
    for (int i = 0; i < 9; ++i) {
        const int Ps = __float2int_rn(Psf[i]);
        eabs += static_cast<unsigned>(Ps);
        a[i] = (Ps & ~15) | (15 - i);
    }
    // |key| < 2^29 + 2^14, so the sum of three keys fits 32 bits: middle = sum - max - min
    const int h1 = __vimax3_s32(a[0], a[1], a[2]), l1 = __vimin3_s32(a[0], a[1], a[2]), d1 = a[0] + a[1] + a[2] - h1 - l1;
    const int h2 = __vimax3_s32(a[3], a[4], a[5]), l2 = __vimin3_s32(a[3], a[4], a[5]), d2 = a[3] + a[4] + a[5] - h2 - l2;
    const int h3 = __vimax3_s32(a[6], a[7], a[8]), l3 = __vimin3_s32(a[6], a[7], a[8]), d3 = a[6] + a[7] + a[8] - h3 - l3;
    const int m1 = __vimax3_s32(h1, h2, h3), lh = __vimin3_s32(h1, h2, h3), mh = h1 + h2 + h3 - m1 - lh;
    const int dmax = __vimax3_s32(d1, d2, d3), lmax = __vimax3_s32(l1, l2, l3);
    const int m2 = max(mh, dmax), B = min(mh, dmax);
    const int m3 = __vimax3_s32(B, lh, lmax);
    // fourth: the runner-up of {B, lh, lmax} or the middle one of the triples' middle keys
    const int dmed = d1 + d2 + d3 - dmax - __vimin3_s32(d1, d2, d3);
    const int m4 = max(B + lh + lmax - m3 - __vimin3_s32(B, lh, lmax), dmed);

    const unsigned t = (eabs & static_cast<unsigned>(kOne - 1)) != 0u ? 1u : 0u;
    const unsigned jx = (eabs - t) >> 29;   // <= 7 for any 32-bit value
    const bool zero = eabs == 0u;   // e == 0: no flips, no candidate
    const int mc = jx <= 1u ? m1 : (jx <= 3u ? m2 : (jx <= 5u ? m3 : m4));
    // |float sum| < 3.75 * 2^30 bounds the true |e| below 0xF0001000; a sum that wrapped because
    // the float sign was wrong is >= 0xFFFFF000
    const bool big = !(fabsf(ef) < 0x1.ep31f) | (eabs >= 0xF8000000u);
    const bool ok = !big & ((mc >= (1 << 27)) | zero);
    // Every key carries the index of a real element, so the positions below are 0..8 whatever
    // the input; ranks 1 and 2 are read-modify-written unconditionally (a zero change when the
    // flip does not apply), ranks 3 and 4 are rare enough for a branch.
    SQ_DBG((~m1 & 15) < 9 && (~m2 & 15) < 9 && (~m3 & 15) < 9 && (~m4 & 15) < 9, 1);   // every key carries a real element's index
    {
        unsigned char *p1 = cb + (~m1 & 15);
        *p1 = static_cast<unsigned char>(*p1 - ((ok & (jx >= 1u)) ? sgn : 0));
        unsigned char *p2 = cb + (~m2 & 15);
        *p2 = static_cast<unsigned char>(*p2 - ((ok & (jx >= 3u)) ? sgn : 0));
    }
    if (ok & (jx >= 5u)) {
        unsigned char *p3 = cb + (~m3 & 15);
        *p3 = static_cast<unsigned char>(*p3 - sgn);
        if (jx == 7u) {
            unsigned char *p4 = cb + (~m4 & 15);
            *p4 = static_cast<unsigned char>(*p4 - sgn);
        }
    }
    const int vs = (mc & ~15) - static_cast<int>((jx & 1u) << 30);   // Over: value after the flip
    const unsigned k = (jx + 1u) >> 1;
    e_out = ok ? sgn * static_cast<int>(eabs - (k << 30)) : 0;
    v_out = (ok & !zero) ? sgn * vs : 0;
    idx_out = ok ? static_cast<unsigned>(~mc & 15) : kRedoMark;
    return !ok;
}

// ---------------------------------------------------------------- one output channel
// Stages output channel m in the group's shared-memory slice, takes its absmax and returns the
// scale (0 if the staging wait ran out: the caller must leave without writing).  A channel that
// starts on a 16-byte boundary and whose length is a multiple of four floats arrives by ONE bulk
// asynchronous copy issued by the group's first thread (the whole channel is in flight at once,
// no registers or load instructions spent on it); anything else is fetched with plain loads.
// Ends with a group barrier, so the staged weights are visible to the whole group.
__device__ __forceinline__ float stage_channel(const LayerDesc &L, int m, const Group &G,
                                               unsigned char *slice, int qmax)
{
    const int NK = L.NK;
    float *wbuf = reinterpret_cast<float *>(slice);
    unsigned char *red = slice + L.off_red;
    unsigned long long *bar = reinterpret_cast<unsigned long long *>(red + 192);
    int *flag = reinterpret_cast<int *>(red + 200);
    const float *wg = L.w + static_cast<size_t>(m) * NK;
    float amax = 0.0f;
    {   // channel-step scratch starts at zero; the barriers below publish it
        int *hist = reinterpret_cast<int *>(slice + L.off_hist);
        for (int i = G.t; i < kHistBins; i += G.g) hist[i] = 0;
        if (G.t == 0) {
            reinterpret_cast<int *>(red + 128)[5] = 0;                    // boundary-list count
            reinterpret_cast<int *>(red + 128)[6] = 0;                    // redo-list count (3x3 fast path)
            *reinterpret_cast<unsigned long long *>(red + 208) = 0ull;   // channel-sum accumulator
            *reinterpret_cast<unsigned *>(red + 216) = 0u;               // absmax slot
        }
    }
    if (G.g == 32 && (reinterpret_cast<uintptr_t>(wg) & 15) == 0 && (NK & 3) == 0) {
        // A channel of at most 1024 weights (one warp): plain 128-bit loads, all issued at once,
        // arrive sooner than a bulk copy that is waited for through an mbarrier.
        const int nv = NK >> 2;
        const float4 *src = reinterpret_cast<const float4 *>(wg);
#pragma unroll 8
        for (int i = G.t; i < nv; i += 32) {
            const float4 t = __ldcs(src + i);
            reinterpret_cast<float4 *>(wbuf)[i] = t;
            amax = fmaxf(fmaxf(amax, fabsf(t.x)), fmaxf(fabsf(t.y), fmaxf(fabsf(t.z), fabsf(t.w))));
        }
        G.sync();   // staged weights and the zeroed scratch are visible
        amax = group_absmax(G, amax, red);
    } else if ((reinterpret_cast<uintptr_t>(wg) & 15) == 0 && (NK & 3) == 0) {
        if (G.t == 0) {   // one thread waits for the copy; the others wait for it at the barrier
            mbar_init(bar, 1);
            bulk_load(wbuf, wg, static_cast<unsigned>(NK) * 4u, bar);
            *flag = mbar_wait(bar, 0) ? 0 : 1;
        }
        G.sync();   // the staged channel (written by the async proxy, observed through the mbarrier) is visible
        const int nv = NK >> 2;
        const float4 *src = reinterpret_cast<const float4 *>(wbuf);
#pragma unroll 3
        for (int i = G.t; i < nv; i += G.g) {
            const float4 t = src[i];
            amax = fmaxf(fmaxf(amax, fabsf(t.x)), fmaxf(fabsf(t.y), fmaxf(fabsf(t.z), fabsf(t.w))));
        }
        amax = group_absmax(G, amax, red);
        if (*flag) {   // group-uniform after the barrier inside group_absmax
            if (G.t == 0) atomicExch(&g_device_status, 1);
            return 0.0f;
        }
    } else {
        for (int i = G.t; i < NK; i += G.g) {
            const float t = __ldcs(wg + i);
            wbuf[i] = t;
            amax = fmaxf(amax, fabsf(t));
        }
        G.sync();   // the zeroed scratch is visible before the reduction uses it
        amax = group_absmax(G, amax, red);
    }
    return (amax < 0x1p-100f) ? 1.0f : __fdiv_rn(amax, static_cast<float>(qmax));
}

// SQuant-C on the staged channel: channel sum, flip count, threshold of the radix select.
struct ChannelStep {
    long long ec;            // channel error sum after SQuant-C
    int sgn_c, k_eff;        // direction and number of kernels to flip (k_eff = 0: none)
    unsigned long long T;    // kernels whose candidate key is >= T are flipped
};

__device__ __forceinline__ ChannelStep channel_step(const LayerDesc &L, const Group &G,
                                                    unsigned char *slice, long long esum,
                                                    unsigned mode)
{
    int *vv = reinterpret_cast<int *>(slice + L.off_vv);
    int *hist = reinterpret_cast<int *>(slice + L.off_hist);
    unsigned char *red = slice + L.off_red;
    int *bc = reinterpret_cast<int *>(red + 128);
    ChannelStep c;
    c.ec = 0; c.sgn_c = 0; c.k_eff = 0; c.T = ~0ull;
    if ((mode & 4u) || L.cerr) c.ec = group_sum(G, esum, red);   // barrier: per-kernel data visible
    else G.sync();
    if ((mode & 4u) && c.ec != 0) {
        c.sgn_c = c.ec > 0 ? 1 : -1;
        const long long abs_e = c.ec > 0 ? c.ec : -c.ec;
        const int kc = static_cast<int>(min((abs_e + (kHalf - 1)) >> 30, 1ll << 30));   // a clipped channel's sum can be huge
        if (kc > 0) c.k_eff = select_threshold(G, vv, L.N, c.sgn_c, kc, hist, bc, c.T);
        c.ec -= static_cast<long long>(c.sgn_c) * c.k_eff * kOne;
    }
    return c;
}

// ---------------------------------------------------------------- emit one channel
// Codes of one channel from the staging buffer to global memory, then scale and channel error.
// Called by the whole group right after a group barrier that made the final staged codes
// visible.  int8: N*K bytes; packed int4 (kModePackInt4 in `mode`, bits <= 4): two codes per byte,
// low nibble = even flat index, ceil(N*K / 2) bytes per output channel, packed into `scratch`
// (shared memory that is dead by now) first.  Aligned rows leave by one bulk asynchronous copy.
constexpr unsigned kModePackInt4 = 0x100u;
constexpr unsigned kModeWideRange = 0x200u;   // the clip range is [-qmax - 1, qmax] (no narrow-range flag)

// fp32 -> bfloat16 (the upper half of the fp32 pattern), round to nearest, ties to even; finite input
__device__ __forceinline__ unsigned bf16_bits(float f)
{
    const unsigned u = __float_as_uint(f);
    return (u + 0x7fffu + ((u >> 16) & 1u)) >> 16;
}

__device__ __forceinline__ void emit_channel(const LayerDesc &L, int m, const Group &G,
                                             const unsigned char *cbuf, unsigned char *scratch, float s,
                                             long long ec, unsigned mode)
{
    const int NK = L.NK;
    if (L.deq16) {   // the same product as bfloat16
        uint16_t *dg = L.deq16 + static_cast<size_t>(m) * NK;
        if ((reinterpret_cast<uintptr_t>(dg) & 7) == 0 && (NK & 3) == 0) {
            for (int i = G.t; i < (NK >> 2); i += G.g) {
                const unsigned c4 = reinterpret_cast<const unsigned *>(cbuf)[i];
                const unsigned b0 = bf16_bits(__fmul_rn(__int2float_rn(static_cast<signed char>(c4 & 255u)), s));
                const unsigned b1 = bf16_bits(__fmul_rn(__int2float_rn(static_cast<signed char>((c4 >> 8) & 255u)), s));
                const unsigned b2 = bf16_bits(__fmul_rn(__int2float_rn(static_cast<signed char>((c4 >> 16) & 255u)), s));
                const unsigned b3 = bf16_bits(__fmul_rn(__int2float_rn(static_cast<signed char>(c4 >> 24)), s));
                __stcs(reinterpret_cast<uint2 *>(dg) + i, make_uint2(b0 | (b1 << 16), b2 | (b3 << 16)));
            }
        } else {
            for (int i = G.t; i < NK; i += G.g)
                dg[i] = static_cast<uint16_t>(bf16_bits(__fmul_rn(__int2float_rn(static_cast<signed char>(cbuf[i])), s)));
        }
    }
    if (L.deq) {   // Algorithm 1's own return value: code * s, fp32
        float *dg = L.deq + static_cast<size_t>(m) * NK;
        if ((reinterpret_cast<uintptr_t>(dg) & 15) == 0 && (NK & 3) == 0) {
            for (int i = G.t; i < (NK >> 2); i += G.g) {
                const unsigned c4 = reinterpret_cast<const unsigned *>(cbuf)[i];
                float4 f;
                f.x = __fmul_rn(__int2float_rn(static_cast<signed char>(c4 & 255u)), s);
                f.y = __fmul_rn(__int2float_rn(static_cast<signed char>((c4 >> 8) & 255u)), s);
                f.z = __fmul_rn(__int2float_rn(static_cast<signed char>((c4 >> 16) & 255u)), s);
                f.w = __fmul_rn(__int2float_rn(static_cast<signed char>(c4 >> 24)), s);
                __stcs(reinterpret_cast<float4 *>(dg) + i, f);
            }
        } else {
            for (int i = G.t; i < NK; i += G.g)
                dg[i] = __fmul_rn(__int2float_rn(static_cast<signed char>(cbuf[i])), s);
        }
    }
    const unsigned char *src = cbuf;
    int row = NK;
    if (mode & kModePackInt4) {
        row = (NK + 1) >> 1;
        const int pairs = NK >> 1;
        for (int i = G.t; i < pairs; i += G.g)
            scratch[i] = static_cast<unsigned char>((cbuf[2 * i] & 15) | (cbuf[2 * i + 1] << 4));
        if ((NK & 1) && G.t == 0) scratch[pairs] = static_cast<unsigned char>(cbuf[NK - 1] & 15);
        G.sync();
        src = scratch;
    }
    unsigned char *cg = reinterpret_cast<unsigned char *>(L.codes) + static_cast<size_t>(m) * row;
    const bool aligned = (reinterpret_cast<uintptr_t>(cg) & 15) == 0;
    const bool bulk = aligned && (row & 15) == 0 && G.g > 32;   // a one-warp group stores its few bytes itself
    if (bulk) {
        if (G.t == 0) bulk_store(cg, src, static_cast<unsigned>(row));
    } else if (aligned) {
        const int nv = row >> 4;
        for (int i = G.t; i < nv; i += G.g) __stcs(reinterpret_cast<int4 *>(cg) + i, reinterpret_cast<const int4 *>(src)[i]);
        for (int i = (nv << 4) + G.t; i < row; i += G.g) cg[i] = src[i];
    } else {
        for (int i = G.t; i < row; i += G.g) cg[i] = src[i];
    }
    if (G.t == 0) {
        L.scales[m] = s;
        if (L.cerr) L.cerr[m] = __fmul_rn(__ll2float_rn(ec), 0x1p-30f);
        if (bulk) bulk_store_wait();   // shared memory must stay intact until the bulk copy has read it
    }
}

// ---------------------------------------------------------------- one kernel by a whole warp
// The same as kernel_generic for a channel with few kernels of many elements (a 7x7 stem has three
// per output channel): thread-per-kernel would leave 29 lanes idle while three walk up to 25
// arg-max rounds over 49 keys each.  Here the warp takes one kernel at a time, lane l holding
// elements l, l + 32, ...: every round is a lane-local scan and three warp reductions (largest
// key, lowest index among its holders).  Called by all 32 lanes; the results are warp-uniform.
__device__ __forceinline__ void kernel_warp(float *wk, int K, float s, bool do_k, int8_t *ck, int lane,
                                            long long &e_out, int &v_out, int &idx_out)
{
    int *Pk = reinterpret_cast<int *>(wk);
    long long e = 0;
    for (int i = lane; i < K; i += 32) {
        int q, P;
        squant_e(wk[i], s, q, P);
        ck[i] = static_cast<int8_t>(q);
        Pk[i] = P;
        e += P;
    }
    {   // |e| <= K / 2 < 2^15 units: hi and lo halves cannot overflow 32 bits over a warp
        const int hi = __reduce_add_sync(kFull, static_cast<int>(e >> 16));
        const int lo = __reduce_add_sync(kFull, static_cast<int>(e & 0xffff));
        e = (static_cast<long long>(hi) << 16) + lo;
    }
    __syncwarp();
    int v = 0, idx = 0;
    if (e != 0) {
        const int sgn = e > 0 ? 1 : -1;
        const long long abs_e = e > 0 ? e : -e;
        const int k = do_k ? flip_count(abs_e) : 0;
        int flips = 0, last = -1, cand = -1;
        for (int r = 0; r <= k; ++r) {
            int best = 0, bi = 0x7fffffff;
            for (int i = lane; i < K; i += 32) {
                const int key = sgn * Pk[i];
                if (key > best) { best = key; bi = i; }   // strict: the lane's lowest index wins its ties
            }
            const int top = __reduce_max_sync(kFull, best);
            if (top <= 0) break;
            const int who = __reduce_min_sync(kFull, best == top ? bi : 0x7fffffff);
            if (r < k) {
                if (who % 32 == lane) {
                    Pk[who] -= sgn * kOne;
                    ck[who] = static_cast<int8_t>(ck[who] - sgn);
                }
                __syncwarp();
                last = who;
                ++flips;
            } else {
                cand = who;
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

// ---------------------------------------------------------------- one whole channel per thread
// Depthwise convolutions: one kernel per output channel (N = 1), so SQuant-C has nothing to do once
// SQuant-K has run (the channel's sum is the kernel's, within one half), and a channel is a handful
// of weights.  One thread takes the whole channel - absmax, scale, SQuant-E/K, stores - and a
// 256-thread CTA takes 256 channels instead of eight.  slice: K floats and K code bytes of the thread.
__device__ __forceinline__ void channel_single(const LayerDesc &L, int m, unsigned char *slice, int qmax, unsigned mode)
{
    const int K = L.K;
    float *wk = reinterpret_cast<float *>(slice);
    int8_t *ck = reinterpret_cast<int8_t *>(slice + 4 * K);
    const float *wg = L.w + static_cast<size_t>(m) * K;
    float amax = 0.0f;
    for (int i = 0; i < K; ++i) {
        const float t = __ldcs(wg + i);
        wk[i] = t;
        amax = fmaxf(amax, fabsf(t));
    }
    const float s = (amax < 0x1p-100f) ? 1.0f : __fdiv_rn(amax, static_cast<float>(qmax));
    long long e;
    int v, idx;
    kernel_generic(wk, K, s, (mode & 2u) != 0, ck, e, v, idx);
    int8_t *cg = L.codes + static_cast<size_t>(m) * K;
    for (int i = 0; i < K; ++i) cg[i] = ck[i];
    const float ef = __fmul_rn(__ll2float_rn(e), 0x1p-30f);
    L.scales[m] = s;
    if (L.kerr) L.kerr[m] = ef;
    if (L.cerr) L.cerr[m] = ef;
}

// ---------------------------------------------------------------- channel body, any kernel size
template <int KT>
__device__ __forceinline__ void channel_body(const LayerDesc &L, int m, const Group &G,
                                             unsigned char *slice, float s, unsigned mode)
{
    const int K = KT ? KT : L.K;
    const int N = L.N;
    float *wbuf = reinterpret_cast<float *>(slice);
    int8_t *cbuf = reinterpret_cast<int8_t *>(slice + L.off_codes);
    int *ev = reinterpret_cast<int *>(slice + L.off_ev);
    int *vv = reinterpret_cast<int *>(slice + L.off_vv);
    unsigned short *vi = reinterpret_cast<unsigned short *>(slice + L.off_vi);

    // ---- SQuant-E, SQuant-K, candidate: one thread per kernel
    // Without SQuant-K a kernel sum can reach K/2 and no longer fits 32 bits; it is then
    // emitted right here (no channel step follows: E|C on larger kernels has its own body).
    const bool do_k = (mode & 2u) != 0;
    const bool keep = do_k || KT == 1 || K == 1;
    float *kerr = L.kerr ? L.kerr + static_cast<size_t>(m) * N : nullptr;
    long long esum = 0;
    if (KT == 0 && K >= 16 && 4 * N <= G.g) {
        // few kernels of many elements: a warp per kernel, lanes over its elements
        const int lane = G.t & 31;
        for (int n = G.t >> 5; n < N; n += G.g >> 5) {
            long long e1;
            int v, idx;
            kernel_warp(wbuf + static_cast<size_t>(n) * K, K, s, do_k, cbuf + static_cast<size_t>(n) * K, lane, e1, v, idx);
            if (lane == 0) {
                if (keep) {
                    ev[n] = static_cast<int>(e1);
                    vv[n] = v;
                    vi[n] = static_cast<unsigned short>(idx);
                } else if (kerr) {
                    kerr[n] = __fmul_rn(__ll2float_rn(e1), 0x1p-30f);
                }
                esum += e1;
            }
        }
    } else
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
    const ChannelStep cs = channel_step(L, G, slice, esum, mode);
    const long long ec = cs.ec;
    const int sgn_c = cs.sgn_c, k_eff = cs.k_eff;
    const unsigned long long T = cs.T;

    // ---- apply the channel flips, emit the kernels' error sums
    if (keep && (k_eff > 0 || kerr)) {
        for (int n = G.t; n < N; n += G.g) {
            int e1 = ev[n];
            if (k_eff > 0) {
                const unsigned long long ck = cand_key(vv[n], sgn_c, n);
                if (ck != 0 && ck >= T) {
                    e1 -= sgn_c * kOne;
                    const size_t j = (KT == 1) ? n : static_cast<size_t>(n) * K + vi[n];
                    if (SQ_DBG_OK(j < static_cast<size_t>(L.NK) && (KT == 1 || vi[n] < K), 2)) cbuf[j] = static_cast<int8_t>(cbuf[j] - sgn_c);
                }
            }
            if (kerr) kerr[n] = __fmul_rn(__int2float_rn(e1), 0x1p-30f);
        }
    }
    G.sync();
#ifdef SQUANT_DEBUG_BOUNDS
    // Checked build, kernels kept in shared memory: the perturbations staged after SQuant-K, summed
    // again, minus one unit per channel flip must equal the channel sum.
    if (KT == 0 && ((mode & 4u) || L.cerr)) {
        const int *Pall = reinterpret_cast<const int *>(slice);
        long long chk = 0;
        for (int j = G.t; j < N * K; j += G.g) chk += Pall[j];
        chk = group_sum(G, chk, slice + L.off_red);
        if (G.t == 0) SQ_DBG(chk - static_cast<long long>(sgn_c) * k_eff * kOne == ec, 9);
    }
#endif

    // ---- codes, scale, channel error (the staged weights / perturbations are dead: scratch)
    emit_channel(L, m, G, reinterpret_cast<const unsigned char *>(cbuf), slice, s, ec, mode);
}

// ---------------------------------------------------------------- channel body, caller-supplied scale
// With a supplied scale the clip of Sec. 2.2 fires, so nothing of what the other bodies assume
// holds: a perturbation can be far beyond one half (it is summed in 64 bits; the 32-bit copy used
// for the selection saturates, which is harmless because a clipped element is no candidate), an
// element at the edge of the range cannot be flipped outward, and a kernel or channel can run
// out of candidates before its sum is within one half.  Plain thread-per-kernel code, any kernel
// size, IEEE division; correctness first.  The layer's slice keeps e', v and idx in arrays of
// their own also for 1x1 kernels (the host lays such layers out that way).
// SQuant-E with the clip, SQuant-K with in-range flips only and the candidate of Algorithm 3 for
// the kernel whose K weights sit at wk (overwritten by the 32-bit perturbations); codes go to ck.
__device__ __forceinline__ void kernel_clip(float *wk, int K, float s, bool do_k, int qmin, int qmax, int8_t *ck,
                                            long long &e_out, int &v_out, int &idx_out)
{
    int *Pk = reinterpret_cast<int *>(wk);
    long long e = 0;
    for (int i = 0; i < K; ++i) {
        const float x = __fdiv_rn(wk[i], s);
        const float qf = fminf(fmaxf(rintf(x), static_cast<float>(qmin)), static_cast<float>(qmax));   // the clip of Sec. 2.2
        const long long P = __float2ll_rn(__fmul_rn(__fsub_rn(qf, x), 1073741824.0f));
        ck[i] = static_cast<int8_t>(__float2int_rn(qf));
        Pk[i] = static_cast<int>(max(min(P, 0x7fffffffll), -0x7fffffffll));
        e += P;
    }
    int v = 0, idx = 0;
    if (e != 0) {
        const int sgn = e > 0 ? 1 : -1;
        const long long abs_e = e > 0 ? e : -e;
        const int k = do_k ? static_cast<int>(min((abs_e + (kHalf - 1)) >> 30, static_cast<long long>(K) + 1)) : 0;
        int flips = 0, last = -1, cand = -1;
        for (int r = 0; r <= k; ++r) {
            int best = 0, bi = -1;
            for (int i = 0; i < K; ++i) {
                const int key = sgn * Pk[i], fl = ck[i] - sgn;
                if (key > best && fl >= qmin && fl <= qmax) { best = key; bi = i; }
            }
            if (bi < 0) break;   // out of candidates: the kernel keeps what is left of its sum
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

__device__ __forceinline__ void channel_body_clip(const LayerDesc &L, int m, const Group &G, unsigned char *slice, float s,
                                                  unsigned mode, int qmax)
{
    const int K = L.K, N = L.N;
    const int qmin = (mode & kModeWideRange) ? -qmax - 1 : -qmax;
    float *wbuf = reinterpret_cast<float *>(slice);
    int8_t *cbuf = reinterpret_cast<int8_t *>(slice + L.off_codes);
    int *ev = reinterpret_cast<int *>(slice + L.off_ev);
    int *vv = reinterpret_cast<int *>(slice + L.off_vv);
    unsigned short *vi = reinterpret_cast<unsigned short *>(slice + L.off_vi);
    const bool do_k = (mode & 2u) != 0;
    float *kerr = L.kerr ? L.kerr + static_cast<size_t>(m) * N : nullptr;
    long long esum = 0;
    for (int n = G.t; n < N; n += G.g) {
        long long e;
        int v, idx;
        kernel_clip(wbuf + static_cast<size_t>(n) * K, K, s, do_k, qmin, qmax, cbuf + static_cast<size_t>(n) * K, e, v, idx);
        // a kernel that SQuant-C can flip has a candidate, hence |e'| <= 1/2: its 32-bit copy is exact
        ev[n] = static_cast<int>(max(min(e, 0x7fffffffll), -0x7fffffffll));
        vv[n] = v;
        vi[n] = static_cast<unsigned short>(idx);
        if (kerr) kerr[n] = __fmul_rn(__ll2float_rn(e), 0x1p-30f);
        esum += e;
    }
    const ChannelStep cs = channel_step(L, G, slice, esum, mode);
    if (cs.k_eff > 0) {
        for (int n = G.t; n < N; n += G.g) {
            const unsigned long long ck = cand_key(vv[n], cs.sgn_c, n);
            if (ck != 0 && ck >= cs.T) {
                const size_t j = static_cast<size_t>(n) * K + vi[n];
                cbuf[j] = static_cast<int8_t>(cbuf[j] - cs.sgn_c);
                if (kerr) kerr[n] = __fmul_rn(__int2float_rn(ev[n] - cs.sgn_c * kOne), 0x1p-30f);
            }
        }
    }
    G.sync();
    emit_channel(L, m, G, reinterpret_cast<const unsigned char *>(cbuf), slice, s, cs.ec, mode);
}

// ---------------------------------------------------------------- channel body, E + C without K
// The E&C ablation of the paper's granularity study (Table 5): SQuant-K is left out, so every
// ELEMENT of the channel is its own candidate for SQuant-C (Algorithm 2 on the channel with the
// elements' perturbations as keys, ties by lower flat index).  The channel is handled as N*K
// one-element kernels (the layer's slice is laid out that way); the kernels' error sums are
// formed afterwards from the final perturbations.
__device__ __forceinline__ void channel_body_ec(const LayerDesc &L, int m, const Group &G,
                                                unsigned char *slice, float s, unsigned mode)
{
    const int N = L.N, K = L.K, NK = L.NK;
    float *wbuf = reinterpret_cast<float *>(slice);
    int *P = reinterpret_cast<int *>(slice);   // perturbations overwrite the weights
    int8_t *cbuf = reinterpret_cast<int8_t *>(slice + L.off_codes);
    int *hist = reinterpret_cast<int *>(slice + L.off_hist);
    unsigned char *red = slice + L.off_red;
    int *bc = reinterpret_cast<int *>(red + 128);
    long long esum = 0;
    for (int j = G.t; j < NK; j += G.g) {
        int q, p;
        squant_e(wbuf[j], s, q, p);
        cbuf[j] = static_cast<int8_t>(q);
        P[j] = p;
        esum += p;
    }
    long long ec = group_sum(G, esum, red);   // barrier: perturbations and codes visible
    if (ec != 0) {
        const int sgn_c = ec > 0 ? 1 : -1;
        const long long abs_e = ec > 0 ? ec : -ec;
        const int kc = flip_count(abs_e);
        if (kc > 0) {
            unsigned long long T = ~0ull;
            const int k_eff = select_threshold(G, P, NK, sgn_c, kc, hist, bc, T);
            ec -= static_cast<long long>(sgn_c) * k_eff * kOne;
            if (k_eff > 0) {
                for (int j = G.t; j < NK; j += G.g) {
                    const unsigned long long ck = cand_key(P[j], sgn_c, j);
                    if (ck != 0 && ck >= T) {
                        P[j] -= sgn_c * kOne;
                        cbuf[j] = static_cast<int8_t>(cbuf[j] - sgn_c);
                    }
                }
            }
        }
    }
    G.sync();
    if (L.kerr) {
        float *kerr = L.kerr + static_cast<size_t>(m) * N;
        for (int n = G.t; n < N; n += G.g) {
            long long e = 0;
            for (int i = 0; i < K; ++i) e += P[n * K + i];
            kerr[n] = __fmul_rn(__ll2float_rn(e), 0x1p-30f);
        }
        G.sync();   // the perturbations are scratch for the packed emit
    }
    emit_channel(L, m, G, reinterpret_cast<const unsigned char *>(cbuf), slice, s, ec, mode);
}

// ---------------------------------------------------------------- SQuant-C by histogram (fast paths)
constexpr int kListCap = 128;   // the boundary list lives in the histogram's 1 KB once the scan is done

__device__ __forceinline__ void hist_add(int *hist, int v)
{
    // |v| < 2^30 for every valid candidate; unsigned arithmetic keeps the bin in range for garbage input too
    const unsigned a = v < 0 ? 0u - static_cast<unsigned>(v) : static_cast<unsigned>(v);
    atomicAdd(&hist[min(a >> 22, static_cast<unsigned>(kHistBins - 1))], (v > 0 ? 1 : 0) | (v < 0 ? 0x10000 : 0));
}

// Second half of a fast-path channel: channel sum, SQuant-C by the candidate histogram, flips,
// patched error sums, stores.  KT = 9: kernel n's candidate byte is cbuf[9 n + vi[n]];
// KT = 1: every element is its own kernel and candidate (vv = ev = the perturbations, byte n).
// Needs N % 4 = 0.
template <int KT>
__device__ __forceinline__ void finish_channel_hist(const LayerDesc &L, int m, const Group &G,
                                                    unsigned char *slice, float s, unsigned mode,
                                                    long long esum, float *kerr, float y, float s2,
                                                    void *w_release = nullptr, unsigned char *pack_scratch = nullptr)
{
    const int N = L.N;
    unsigned char *cbuf = slice + L.off_codes;
    int *ev = reinterpret_cast<int *>(slice + L.off_ev);
    int *vv = reinterpret_cast<int *>(slice + L.off_vv);
    unsigned char *vi = slice + L.off_vi;
    int *hist = reinterpret_cast<int *>(slice + L.off_hist);
    unsigned char *red = slice + L.off_red;
    int *bc = reinterpret_cast<int *>(red + 128);               // [0..3] scan result, [5] list count
    unsigned long long *acc = reinterpret_cast<unsigned long long *>(red + 208);
    int2 *blist = reinterpret_cast<int2 *>(slice + L.off_hist); // boundary list: reuses the histogram after the scan
    const int quads = N >> 2;
    // channel sum: two 32-bit warp reductions (|esum| < 2^40 per thread, so the halves cannot
    // overflow over 32 lanes), then one shared atomic per warp
    {
        const int hi = __reduce_add_sync(kFull, static_cast<int>(esum >> 16));
        const int lo = __reduce_add_sync(kFull, static_cast<int>(esum & 0xffff));
        if ((G.t & 31) == 0)
            atomicAdd(acc, static_cast<unsigned long long>((static_cast<long long>(hi) << 16) + lo));
    }
    G.sync();   // per-kernel data, histogram, channel sum and redo list visible
    if (KT == 9) {
        // Kernels the fast selection reported: redone exactly from the staged weights, one
        // thread per kernel.  The list holds N / 2 entries; beyond that (inputs made of ties or
        // of weights tiny against the channel's scale) every thread redoes its own marked kernels.
        const int cnt = bc[6];
        if (cnt > 0) {   // group-uniform
            const float *wbuf = reinterpret_cast<const float *>(slice);
            const unsigned short *redo = reinterpret_cast<const unsigned short *>(vi + N);
            const bool listed = cnt <= (N >> 1);
            const int end = listed ? cnt : N;
            for (int i = G.t; i < end; i += G.g) {
                int n = i;
                if (listed) n = redo[i];
                else if (vi[i] != kRedoMark) continue;
                const KernelOut o = kernel9_exact(wbuf + n * 9, y, s2, cbuf + n * 9);
                ev[n] = o.e;
                vv[n] = o.v;
                vi[n] = static_cast<unsigned char>(o.idx);
                if (kerr) kerr[n] = __fmul_rn(__int2float_rn(o.e), 0x1p-30f);
                if (o.v != 0) hist_add(hist, o.v);
                atomicAdd(acc, static_cast<unsigned long long>(static_cast<long long>(o.e)));
            }
            G.sync();
        }
        // the staged weights are dead from here on: a pipelined caller lets the next copy start
        if (w_release != nullptr && G.t == 0) mbar_arrive(w_release);
    }
    long long ec = static_cast<long long>(*acc);

    // ---- SQuant-C: boundary bin of the candidate histogram
    int sgn_c = 0, k_eff = 0;
    int t_all = 0x7fffffff;     // candidates with v * sgn_c >= t_all are flipped outright
    int t_list = 0x7fffffff;    // those in [t_list, t_all) go to the boundary list
    int rem = 0, cb = 0;
    unsigned long long T64 = ~0ull;
    bool wide = false;          // fallback: compare 48-bit keys against T64
    if ((mode & 4u) && ec != 0) {
        sgn_c = ec > 0 ? 1 : -1;
        const long long abs_e = ec > 0 ? ec : -ec;
        const int kc = flip_count(abs_e);
        if (kc > 0) {
            if (G.t < 32) {   // the group's first warp scans, highest bins first
                const int lane = G.t, grp = 31 - lane, sh = sgn_c > 0 ? 0 : 16;
                const int4 h0 = reinterpret_cast<const int4 *>(hist)[2 * grp];
                const int4 h1 = reinterpret_cast<const int4 *>(hist)[2 * grp + 1];
                const int c[8] = {(h0.x >> sh) & 0xffff, (h0.y >> sh) & 0xffff, (h0.z >> sh) & 0xffff, (h0.w >> sh) & 0xffff,
                                  (h1.x >> sh) & 0xffff, (h1.y >> sh) & 0xffff, (h1.z >> sh) & 0xffff, (h1.w >> sh) & 0xffff};
                const int s8 = ((c[0] + c[1]) + (c[2] + c[3])) + ((c[4] + c[5]) + (c[6] + c[7]));
                int incl = s8;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int t = __shfl_up_sync(kFull, incl, o);
                    if (lane >= o) incl += t;
                }
                const int total = __shfl_sync(kFull, incl, 31);
                const int wnt = min(kc, total);
                const unsigned bal = __ballot_sync(kFull, incl >= wnt);
                if (wnt <= 0) {
                    if (lane == 0) { bc[0] = -1; bc[1] = 0; bc[2] = 0; bc[3] = 0; }
                } else if (lane == __ffs(bal) - 1) {
                    int bb = -1, cnt = 0, cum = incl - s8;
#pragma unroll
                    for (int j = 7; j >= 0; --j) {
                        if (bb < 0) {
                            if (cum + c[j] >= wnt) { bb = grp * 8 + j; cnt = c[j]; }
                            else cum += c[j];
                        }
                    }
                    bc[0] = bb; bc[1] = wnt - cum; bc[2] = cnt; bc[3] = wnt;
                }
            }
            G.sync();
            const int b = bc[0], want = bc[3];
            rem = bc[1];
            cb = bc[2];
            k_eff = want;
            if (want > 0) {
                if (cb == rem) {                 // whole boundary bin flipped
                    t_all = max(b << 22, 1);     // 0 is "no candidate"
                } else if (cb <= kListCap) {     // rank the boundary bin exactly
                    t_all = (b + 1) << 22;       // b + 1 = 256 gives 2^30, above every |v|
                    t_list = max(b << 22, 1);
                } else {                         // crowded bin: general radix select on 48-bit keys
                    wide = true;
                    G.sync();                    // everyone has read the scan result
                    k_eff = select_threshold(G, vv, N, sgn_c, kc, hist, bc, T64);
                }
            }
            ec -= static_cast<long long>(sgn_c) * k_eff * kOne;
        }
    }

    // ---- flip the selected kernels' candidates and patch their error sums (rare per kernel)
    const bool listing = t_list != 0x7fffffff;
    if (k_eff > 0) {
        const int t_min = wide ? 1 : min(t_all, t_list);
        for (int Q = G.t; Q < quads; Q += G.g) {
            const int4 v4 = reinterpret_cast<const int4 *>(vv)[Q];
            const int v[4] = {v4.x, v4.y, v4.z, v4.w};
            if (max(max(v[0] * sgn_c, v[1] * sgn_c), max(v[2] * sgn_c, v[3] * sgn_c)) < t_min) continue;
#pragma unroll
            for (int kq = 0; kq < 4; ++kq) {
                const int a = v[kq] * sgn_c;
                if (a >= t_min) {
                    const int n = 4 * Q + kq;
                    bool take;
                    if (wide) {
                        take = cand_key(v[kq], sgn_c, n) >= T64;
                    } else {
                        take = a >= t_all;
                        if (!take) {
                            const int pos = atomicAdd(&bc[5], 1);
                            if (pos < kListCap) blist[pos] = make_int2(a, n);
                        }
                    }
                    if (take) {
                        SQ_DBG(n < N && (KT == 1 || vi[n] < 9), 3);
                        unsigned char *bp = cbuf + (KT == 1 ? n : n * 9 + vi[n]);
                        *bp = static_cast<unsigned char>(*bp - sgn_c);
                        if (kerr) kerr[n] = __fmul_rn(__int2float_rn(ev[n] - sgn_c * kOne), 0x1p-30f);
                    }
                }
            }
        }
    }
    G.sync();
    if (listing) {   // exact rank inside the boundary bin: cb entries, the first `rem` are flipped
        for (int i = G.t; i < cb; i += G.g) {
            const int2 me = blist[i];
            int rank = 0;
            for (int j = 0; j < cb; ++j) {
                const int2 o = blist[j];
                rank += (o.x > me.x || (o.x == me.x && o.y < me.y)) ? 1 : 0;
            }
            if (rank < rem) {
                SQ_DBG(me.y >= 0 && me.y < N && cb <= kListCap, 4);
                unsigned char *bp = cbuf + (KT == 1 ? me.y : me.y * 9 + vi[me.y]);
                *bp = static_cast<unsigned char>(*bp - sgn_c);
                if (kerr) kerr[me.y] = __fmul_rn(__int2float_rn(ev[me.y] - sgn_c * kOne), 0x1p-30f);
            }
        }
        G.sync();
    }

#ifdef SQUANT_DEBUG_BOUNDS
    // Checked build, grouped kernel, 3x3: the staged weights are still there, so the channel's error
    // sum can be taken again from scratch - plain IEEE division of every weight, perturbation of
    // its FINAL code - and must equal what the selection machinery arrived at.
    if (KT == 9 && w_release == nullptr && pack_scratch == nullptr) {
        G.sync();
        const float *wchk = reinterpret_cast<const float *>(slice);
        long long chk = 0;
        for (int j = G.t; j < 9 * N; j += G.g) {
            // rounded code and its perturbation (that difference is exact), then whole steps for the flips
            const float x = __fdiv_rn(wchk[j], s), q0 = rintf(x);
            const long long P0 = __float2ll_rn(__fmul_rn(__fsub_rn(q0, x), 1073741824.0f));
            chk += P0 + (static_cast<long long>(static_cast<signed char>(cbuf[j])) - __float2int_rn(q0)) * kOne;
        }
        chk = group_sum(G, chk, red);
        if (G.t == 0) SQ_DBG(chk == ec, 8);
    }
#endif
    // ---- codes, scale, channel error (the staged weights / perturbations are dead: scratch)
    emit_channel(L, m, G, cbuf, pack_scratch ? pack_scratch : slice, s, ec, mode);
}

// ---------------------------------------------------------------- channel body, 3x3 fast path
// Needs K = 9, N a multiple of 4, SQuant-K in the mode mask and 2^-60 <= s <= 2^60.
// A thread owns four consecutive kernels = 36 consecutive weights: nine conflict-free 128-bit
// shared loads in, nine conflict-free 32-bit stores of packed code bytes out; flips are byte
// read-modify-writes on the staged codes.  Kernel error sums are written as soon as SQuant-K is
// done; SQuant-C later patches the few kernels it flips.
//
// SQuant-C needs ONE histogram, filled while the kernels are processed: bin = |v| >> 22 of each
// kernel's candidate, positive and negative candidates counted in the two halves of one 32-bit
// word.  Once the channel sum (hence the sign and k_c) is known, one warp scans the histogram
// of that sign for the boundary bin;
// kernels above it are flipped, the few inside it are collected in a list and ranked exactly
// (|v| descending, kernel index ascending).  A boundary bin too crowded for the list (massive
// ties) falls back to the general radix select.
__device__ __forceinline__ long long k9_quantize(const LayerDesc &L, int m, const Group &G,
                                                 unsigned char *slice, float s, float s2, float y)
{
    const int N = L.N;
    const float *wbuf = reinterpret_cast<const float *>(slice);
    unsigned char *cbuf = slice + L.off_codes;
    int *ev = reinterpret_cast<int *>(slice + L.off_ev);
    int *vv = reinterpret_cast<int *>(slice + L.off_vv);
    unsigned char *vi = slice + L.off_vi;
    int *hist = reinterpret_cast<int *>(slice + L.off_hist);
    float *kerr = L.kerr ? L.kerr + static_cast<size_t>(m) * N : nullptr;
    const bool kvec = (reinterpret_cast<uintptr_t>(kerr) & 15) == 0;

    (void)s;
    const int quads = N >> 2;
    int *redo_cnt = reinterpret_cast<int *>(slice + L.off_red + 128) + 6;
    unsigned short *redo = reinterpret_cast<unsigned short *>(vi + N);   // upper half of the index area
    const int redo_cap = N >> 1;
    long long esum = 0;
    const E2 c2 = make_e2(y, s2);
    for (int Q = G.t; Q < quads; Q += G.g) {
        const float4 *src = reinterpret_cast<const float4 *>(wbuf) + Q * 9;
        unsigned *dst = reinterpret_cast<unsigned *>(cbuf) + Q * 9;
        float2 P2[18];   // the quad's 36 perturbations, pair p = elements 2p, 2p + 1
#pragma unroll
        for (int j = 0; j < 9; ++j) {
            const float4 w = src[j];
            float2 ta, tb;
            squant_e_fast2(make_float2(w.x, w.y), c2, ta, P2[2 * j]);
            squant_e_fast2(make_float2(w.z, w.w), c2, tb, P2[2 * j + 1]);
            dst[j] = __byte_perm(__byte_perm(__float_as_uint(ta.x), __float_as_uint(ta.y), 0x0040),
                                 __byte_perm(__float_as_uint(tb.x), __float_as_uint(tb.y), 0x0040), 0x5410);
        }
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
        int e4[4], v4[4];
        unsigned i4 = 0;
        unsigned char *cq = cbuf + Q * 36;
#pragma unroll
        for (int kq = 0; kq < 4; ++kq) {
            float Pk[9];
#pragma unroll
            for (int i = 0; i < 9; ++i) {
                const int el = 9 * kq + i;
                Pk[i] = (el & 1) ? P2[el >> 1].y : P2[el >> 1].x;
            }
            unsigned idx;
            if (kernel9_select(Pk, ef[kq], cq + 9 * kq, e4[kq], v4[kq], idx)) {   // rare: redone exactly later
                const int pos = atomicAdd(redo_cnt, 1);
                if (pos < redo_cap) redo[pos] = static_cast<unsigned short>(4 * Q + kq);
            }
            {   // candidate histogram; |v| < 2^30 for valid input, the mask keeps garbage in range (v = 0 adds nothing)
                const int v = v4[kq];
                atomicAdd(&hist[(abs(v) >> 22) & (kHistBins - 1)], v > 0 ? 1 : ((v >> 31) & 0x10000));
            }
            i4 |= idx << (8 * kq);
        }
        esum += static_cast<long long>(e4[0] + e4[1]) + (e4[2] + e4[3]);   // pairs fit 32 bits
        reinterpret_cast<int4 *>(ev)[Q] = make_int4(e4[0], e4[1], e4[2], e4[3]);
        reinterpret_cast<int4 *>(vv)[Q] = make_int4(v4[0], v4[1], v4[2], v4[3]);
        reinterpret_cast<unsigned *>(vi)[Q] = i4;
        if (kerr) {
            float4 f;
            f.x = __fmul_rn(__int2float_rn(e4[0]), 0x1p-30f);
            f.y = __fmul_rn(__int2float_rn(e4[1]), 0x1p-30f);
            f.z = __fmul_rn(__int2float_rn(e4[2]), 0x1p-30f);
            f.w = __fmul_rn(__int2float_rn(e4[3]), 0x1p-30f);
            if (kvec) __stcs(reinterpret_cast<float4 *>(kerr) + Q, f);
            else { kerr[4 * Q] = f.x; kerr[4 * Q + 1] = f.y; kerr[4 * Q + 2] = f.z; kerr[4 * Q + 3] = f.w; }
        }
    }
    return esum;
}

__device__ __forceinline__ void channel_body_k9_fast(const LayerDesc &L, int m, const Group &G,
                                                     unsigned char *slice, float s, unsigned mode)
{
    const float s2 = __fmul_rn(s, 0x1p-30f);
    const float y = __frcp_rn(s2);
    const long long esum = k9_quantize(L, m, G, slice, s, s2, y);
    float *kerr = L.kerr ? L.kerr + static_cast<size_t>(m) * L.N : nullptr;
    finish_channel_hist<9>(L, m, G, slice, s, mode, esum, kerr, y, s2);
}

// ---------------------------------------------------------------- channel body, 1x1 fast path
// Fully connected and pointwise layers (K = 1; needs N % 4 = 0 and 2^-60 <= s <= 2^60).  Every
// element is its own kernel, SQuant-K is a no-op (Sec. 3.4) and the element's perturbation is its
// own candidate for SQuant-C.  A thread takes four elements at a time: one 128-bit shared load,
// the reciprocal-based SQuant-E (packed fp32x2), one packed word of codes, and the four integer perturbations
// written back in place of the weights (they are the e' / v arrays of the channel step).
__device__ __forceinline__ void channel_body_k1_fast(const LayerDesc &L, int m, const Group &G,
                                                     unsigned char *slice, float s, unsigned mode)
{
    const int N = L.N;
    float4 *wbuf4 = reinterpret_cast<float4 *>(slice);
    unsigned *cbuf32 = reinterpret_cast<unsigned *>(slice + L.off_codes);
    int *hist = reinterpret_cast<int *>(slice + L.off_hist);
    float *kerr = L.kerr ? L.kerr + static_cast<size_t>(m) * N : nullptr;
    const bool kvec = (reinterpret_cast<uintptr_t>(kerr) & 15) == 0;
    const float s2 = __fmul_rn(s, 0x1p-30f);
    const float y = __frcp_rn(s2);
    const int quads = N >> 2;
    const E2 c2 = make_e2(y, s2);
    long long esum = 0;
    for (int Q = G.t; Q < quads; Q += G.g) {
        const float4 w = wbuf4[Q];
        float2 ta, tb, Pa, Pb;
        squant_e_fast2(make_float2(w.x, w.y), c2, ta, Pa);
        squant_e_fast2(make_float2(w.z, w.w), c2, tb, Pb);
        const int4 P = make_int4(__float2int_rn(Pa.x), __float2int_rn(Pa.y), __float2int_rn(Pb.x), __float2int_rn(Pb.y));
        cbuf32[Q] = __byte_perm(__byte_perm(__float_as_uint(ta.x), __float_as_uint(ta.y), 0x0040),
                                __byte_perm(__float_as_uint(tb.x), __float_as_uint(tb.y), 0x0040), 0x5410);
        reinterpret_cast<int4 *>(wbuf4)[Q] = P;
        if (mode & 4u) {
            hist_add(hist, P.x);
            hist_add(hist, P.y);
            hist_add(hist, P.z);
            hist_add(hist, P.w);
        }
        esum += static_cast<long long>(P.x + P.y) + (P.z + P.w);   // pairs fit 32 bits
        if (kerr) {
            float4 f;
            f.x = __fmul_rn(__int2float_rn(P.x), 0x1p-30f);
            f.y = __fmul_rn(__int2float_rn(P.y), 0x1p-30f);
            f.z = __fmul_rn(__int2float_rn(P.z), 0x1p-30f);
            f.w = __fmul_rn(__int2float_rn(P.w), 0x1p-30f);
            if (kvec) __stcs(reinterpret_cast<float4 *>(kerr) + Q, f);
            else { kerr[4 * Q] = f.x; kerr[4 * Q + 1] = f.y; kerr[4 * Q + 2] = f.z; kerr[4 * Q + 3] = f.w; }
        }
    }
    finish_channel_hist<1>(L, m, G, slice, s, mode, esum, kerr, y, s2);
}

// ---------------------------------------------------------------- self-check of the fast division
// For each given scale s (in the fast path's range) and EVERY fp32 bit pattern w with
// |w| <= s * qmax * (1 + 2^-20) - a superset of what a channel with that scale can contain -
// compares code and integer perturbation from the reciprocal-based SQuant-E, in its scalar and in
// its packed fp32x2 form, with those from the plain IEEE division.  mismatches[i] counts the
// disagreements for scales[i].
__global__ void selfcheck_division_kernel(const float *scales, int n, int qmax,
                                          unsigned long long *mismatches)
{
    const int si = blockIdx.y;
    if (si >= n) return;
    const float s = scales[si];
    const float s2 = __fmul_rn(s, 0x1p-30f);
    const float y = __frcp_rn(s2);
    const float lim = __fmul_rn(__fmul_rn(s, static_cast<float>(qmax)), 1.000001f);
    const E2 c2 = make_e2(y, s2);
    unsigned long long bad = 0;
    const unsigned long long half = 1ull << 31;   // a pair = (w, -w): both lanes of the packed sequence
    for (unsigned long long b = blockIdx.x * static_cast<unsigned long long>(blockDim.x) + threadIdx.x; b < half;
         b += static_cast<unsigned long long>(gridDim.x) * blockDim.x) {
        const float w = __uint_as_float(static_cast<unsigned>(b));
        if (!(w <= lim)) continue;   // also skips NaN
        const float wp[2] = {w, -w};
        float2 t2, P2;
        squant_e_fast2(make_float2(wp[0], wp[1]), c2, t2, P2);
        const float tl[2] = {t2.x, t2.y}, Pl[2] = {P2.x, P2.y};
#pragma unroll
        for (int l = 0; l < 2; ++l) {
            unsigned tb;
            int P_fast, q, P;
            squant_e_fast(wp[l], y, s2, tb, P_fast);   // the scalar sequence (used by the exact redo)
            squant_e(wp[l], s, q, P);                   // plain IEEE division
            const int qs = static_cast<int>(static_cast<signed char>(tb & 255u));
            const int qp = static_cast<int>(static_cast<signed char>(__float_as_uint(tl[l]) & 255u));
            bad += (qs != q) | (P_fast != P) | (qp != q) | (__float2int_rn(Pl[l]) != P);
        }
    }
    for (int o = 16; o > 0; o >>= 1) bad += __shfl_xor_sync(kFull, bad, o);
    if ((threadIdx.x & 31) == 0 && bad) atomicAdd(mismatches + si, bad);
}

// ---------------------------------------------------------------- the bounded wait, on its own
// Waits for a barrier at which nobody ever arrives, with a small poll limit: the wait runs out,
// the thread records it in the status word exactly as the solver kernels do, and the kernel ends.
__global__ void debug_wait_kernel(int max_polls)
{
    __shared__ unsigned long long bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        if (!mbar_wait(&bar, 0u, max_polls)) atomicExch(&g_device_status, 1);
    }
}

// ---------------------------------------------------------------- grouped launch
// One CTA per work item.  The descriptor of the CTA's layer comes either from the launch table
// in the kernel's parameter space (kParams) or from a table in global memory.
#ifndef SQ_MIN_CTAS
#define SQ_MIN_CTAS 4
#endif
__device__ __forceinline__ void run_item(const LayerDesc &L, int ch0, unsigned char *smem, int qmax,
                                         unsigned mode)
{
    if (L.g == 1) {   // depthwise: one channel per thread
        const int m1 = ch0 + static_cast<int>(threadIdx.x);
        if (m1 < L.M) channel_single(L, m1, smem + static_cast<size_t>(threadIdx.x) * L.slice_bytes, qmax, mode);
        return;
    }
    Group G;
    G.g = L.g;
    G.t = threadIdx.x & (L.g - 1);
    const int gi = threadIdx.x >> L.g_shift;
    G.bar = 1 + gi;
    const int m = ch0 + gi;
    if (m >= L.M) return;   // the whole group leaves together; it shares no barrier with others
    unsigned char *slice = smem + static_cast<size_t>(gi) * L.slice_bytes;
    SQ_DBG(ch0 >= 0 && L.g >= 32 && (L.g & (L.g - 1)) == 0 && (1 << L.g_shift) == L.g, 5);
    SQ_DBG(static_cast<size_t>(gi + 1) * L.slice_bytes <= dynamic_smem_bytes(), 6);
    SQ_DBG(L.off_red + 256 <= L.slice_bytes && L.off_hist + 4 * kHistBins <= L.off_red && L.off_codes + L.NK <= L.slice_bytes, 7);
    const float s = stage_channel(L, m, G, slice, qmax);
    if (s == 0.0f) return;   // staging wait ran out (status word set); nothing is written
    if (L.sin) {   // Algorithm 1 with its scale as an input
        float sc = L.sin[m];
        if (!(sc > 0.0f && sc < __int_as_float(0x7f800000))) sc = 1.0f;
        channel_body_clip(L, m, G, slice, sc, mode, qmax);
    } else if (L.K > 1 && (mode & 6u) == 4u) {   // E + C without K
        channel_body_ec(L, m, G, slice, s, mode);
    } else if (L.K == 1) {
        if ((L.N & 3) == 0 && s >= 0x1p-60f && s <= 0x1p60f)
            channel_body_k1_fast(L, m, G, slice, s, mode);
        else
            channel_body<1>(L, m, G, slice, s, mode);
    } else if (L.K == 9) {
        if ((L.N & 3) == 0 && (mode & 2u) && s >= 0x1p-60f && s <= 0x1p60f)
            channel_body_k9_fast(L, m, G, slice, s, mode);
        else
            channel_body<9>(L, m, G, slice, s, mode);
    } else {
        channel_body<0>(L, m, G, slice, s, mode);
    }
}

__global__ void __launch_bounds__(kCtaThreads, SQ_MIN_CTAS)
squant_model_kernel(const __grid_constant__ LaunchTable tbl, int qmax, unsigned mode)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const int item = blockIdx.x;
    int layer = 0;   // uniform binary search for the last layer whose first item is <= item
#pragma unroll 1
    for (int step = tbl.top_step; step > 0; step >>= 1)
        if (layer + step < tbl.n_layers && tbl.first_item[layer + step] <= item) layer += step;
    const LayerDesc &L = tbl.layers[layer];
    const int ch0 = (item - tbl.first_item[layer]) * (kCtaThreads >> L.g_shift);
    run_item(L, ch0, smem, qmax, mode);
}

// The same with the descriptors in a table in global memory (used by the entry point whose
// table lives in a fixed device array).
__global__ void __launch_bounds__(kCtaThreads, SQ_MIN_CTAS)
squant_table_kernel(const LayerDesc *__restrict__ layers, const Item *__restrict__ items, int qmax,
                    unsigned mode)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const Item it = items[blockIdx.x];
    const LayerDesc L = layers[it.layer];
    run_item(L, it.ch0, smem, qmax, mode);
}

}  // namespace sq
