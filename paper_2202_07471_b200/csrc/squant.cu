// Host side of the SQuant library: validation, launch plans, the C ABI of include/squant.h.
#include "squant.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <list>
#include <mutex>
#include <string>
#include <vector>

#include "squant_device.cuh"
#include "squant_pipe.cuh"
#include "squant_stream.cuh"
#include "squant_wide.cuh"

namespace {

using sq::Item;
using sq::LayerDesc;

constexpr int kMaxSmemFallback = 232448;   // 227 KB: per-CTA opt-in limit of sm_100
constexpr int64_t kMaxChannelElems = 65535; // one-CTA paths: keeps the clamp-edge element out of every top-k (its
                                            // perturbation is <= one ulp of qmax); wider channels take the cluster
                                            // kernel, which checks every candidate against the clip range
constexpr int64_t kMaxKernels = (1 << sq::kIdxBits) - 1;   // kernels per channel: the select keys hold 18 index bits
constexpr size_t kMaxPlans = 64;

std::mutex g_mutex;
std::atomic<int64_t> g_launches{0};
thread_local std::string t_cuda_error;

int cuda_fail(cudaError_t e, const char *what)
{
    t_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
    return SQUANT_ERR_CUDA;
}

#define SQ_CUDA(call)                                          \
    do {                                                       \
        cudaError_t e__ = (call);                              \
        if (e__ != cudaSuccess) return cuda_fail(e__, #call);  \
    } while (0)

inline int align16(int v) { return (v + 15) & ~15; }

struct HostPlan {
    std::vector<LayerDesc> layers;
    std::vector<Item> items;
    int smem_bytes = 0;
    int qmax = 0;
    unsigned mode = 0;
};

// Threads that share one output channel, by channel length.
int group_size(int64_t nk)
{
    if (nk <= 1024) return 32;
    if (nk <= 2048) return 64;
    if (nk <= 4096) return 128;
    return 256;
}

int validate(const squant_layer *layers, int32_t n_layers, const squant_options *opt,
             bool need_pointers, squant_options &o)
{
    o.bits = 4;
    o.mode = SQUANT_MODE_EKC;
    o.flags = SQUANT_FLAG_NARROW_RANGE;
    if (opt) {
        o = *opt;
        if (o.mode == 0) o.mode = SQUANT_MODE_EKC;
    }
    if (n_layers < 0) return SQUANT_ERR_SHAPE;
    if (n_layers > 0 && !layers) return SQUANT_ERR_NULL;
    if (o.bits < 2 || o.bits > 8) return SQUANT_ERR_BITS;
    if (!(o.mode & SQUANT_MODE_E) || (o.mode & ~SQUANT_MODE_EKC)) return SQUANT_ERR_MODE;
    if (o.flags & ~(SQUANT_FLAG_NARROW_RANGE | SQUANT_FLAG_PACK_INT4)) return SQUANT_ERR_MODE;
    if ((o.flags & SQUANT_FLAG_PACK_INT4) && o.bits > 4) return SQUANT_ERR_BITS;
    for (int i = 0; i < n_layers; ++i) {
        const squant_layer &l = layers[i];
        if (l.cout <= 0 || l.cin <= 0 || l.kh <= 0 || l.kw <= 0) return SQUANT_ERR_SHAPE;
        const int64_t k = static_cast<int64_t>(l.kh) * l.kw;
        const int64_t nk = k * l.cin;
        if (k > 65535 || nk > (1ll << 30)) return SQUANT_ERR_SHAPE;
        if (static_cast<int64_t>(l.cout) * nk > (1ll << 40)) return SQUANT_ERR_SHAPE;
        if (l.cin > kMaxKernels) return SQUANT_ERR_TOO_WIDE;
        if (need_pointers) {
            if (!l.w || !l.codes || !l.scales) return SQUANT_ERR_NULL;
            if ((reinterpret_cast<uintptr_t>(l.w) & 3) || (reinterpret_cast<uintptr_t>(l.scales) & 3) ||
                (reinterpret_cast<uintptr_t>(l.kernel_err) & 3) ||
                (reinterpret_cast<uintptr_t>(l.channel_err) & 3) || (reinterpret_cast<uintptr_t>(l.dequant) & 3) ||
                (reinterpret_cast<uintptr_t>(l.scales_in) & 3) || (reinterpret_cast<uintptr_t>(l.dequant_bf16) & 1))
                return SQUANT_ERR_ALIGN;
        }
        // supplied scales: the element-wise channel step of E|C on larger kernels is not built for clipping
        if (l.scales_in && k > 1 && (o.mode & SQUANT_MODE_C) && !(o.mode & SQUANT_MODE_K)) return SQUANT_ERR_MODE;
    }
    return SQUANT_OK;
}

// Device-side descriptor of one layer: group size and the layout of a group's shared-memory
// slice.  Returns the dynamic shared memory one CTA needs for this layer.
int64_t layout_layer(const squant_layer &l, LayerDesc &d, unsigned mode, unsigned flags)
{
    d.w = l.w; d.codes = l.codes; d.scales = l.scales; d.kerr = l.kernel_err; d.cerr = l.channel_err; d.deq = l.dequant;
    d.sin = l.scales_in; d.deq16 = l.dequant_bf16;
    d.M = l.cout; d.N = l.cin; d.K = l.kh * l.kw; d.NK = d.N * d.K;
    d.g = group_size(d.NK);
    d.g_shift = 0;
    while ((1 << d.g_shift) < d.g) ++d.g_shift;
    // Depthwise layers (one kernel per output channel) with plain outputs: a whole channel per thread.
    // SQuant-C is void there once SQuant-K has run; without K (E|C) the channel step is real.
    if (d.N == 1 && d.K <= 64 && !l.scales_in && !l.dequant && !l.dequant_bf16 && !(flags & SQUANT_FLAG_PACK_INT4) &&
        ((mode & SQUANT_MODE_K) || !(mode & SQUANT_MODE_C))) {
        d.g = 1;
        d.g_shift = 0;
        d.off_codes = 4 * d.K; d.off_ev = 0; d.off_vv = 0; d.off_vi = 0; d.off_hist = 0; d.off_red = 0;
        d.slice_bytes = align16(5 * d.K);
        return static_cast<int64_t>(sq::kCtaThreads) * d.slice_bytes;
    }
    int off = align16(4 * d.NK);              // staged weights
    d.off_codes = off; off += align16(d.NK);  // staged codes
    const bool ec_only = (mode & SQUANT_MODE_C) && !(mode & SQUANT_MODE_K);   // elements are the candidates
    if ((d.K == 1 || ec_only) && !l.scales_in) {   // perturbations overwrite the weights
        d.off_ev = 0; d.off_vv = 0; d.off_vi = 0;
    } else {
        d.off_ev = off; off += align16(4 * d.N);
        d.off_vv = off; off += align16(4 * d.N);
        d.off_vi = off; off += align16(2 * d.N);
    }
    d.off_hist = off; off += 4 * sq::kHistBins;
    d.off_red = off; off += 256;
    d.slice_bytes = off;
    return static_cast<int64_t>(sq::kCtaThreads / d.g) * off;
}

// Work list in a table (global-memory variant): CTA-sized items, heaviest first.
int build_plan(const squant_layer *layers, int32_t n_layers, const squant_options &o, int max_smem,
               HostPlan &p)
{
    p.qmax = (1 << (o.bits - 1)) - 1;
    p.mode = o.mode | ((o.flags & SQUANT_FLAG_PACK_INT4) ? sq::kModePackInt4 : 0u) |
             ((o.flags & SQUANT_FLAG_NARROW_RANGE) ? 0u : sq::kModeWideRange);
    p.layers.resize(n_layers);
    p.smem_bytes = 0;
    struct Batch { int64_t work; int layer; int ch0; };
    std::vector<Batch> batches;
    for (int i = 0; i < n_layers; ++i) {
        LayerDesc &d = p.layers[i];
        const int64_t cta_smem = layout_layer(layers[i], d, o.mode, o.flags);
        const int groups = sq::kCtaThreads / d.g;
        if (cta_smem > max_smem) return SQUANT_ERR_TOO_WIDE;
        if (cta_smem > p.smem_bytes) p.smem_bytes = static_cast<int>(cta_smem);
        for (int c = 0; c < d.M; c += groups) {
            const int nch = (d.M - c < groups) ? d.M - c : groups;
            batches.push_back({static_cast<int64_t>(nch) * d.NK, i, c});
        }
    }
    // Heaviest CTAs first, so that the tail of the launch is made of light ones.
    std::stable_sort(batches.begin(), batches.end(),
                     [](const Batch &a, const Batch &b) { return a.work > b.work; });
    p.items.resize(batches.size());
    for (size_t i = 0; i < batches.size(); ++i) p.items[i] = {batches[i].layer, batches[i].ch0};
    return SQUANT_OK;
}

// Launch tables for the parameter-space variant: layers ordered by the work of one of their
// CTAs (heaviest first, so the tail of the launch is made of light CTAs), at most
// kMaxParamLayers per launch.
struct ParamPlan {
    std::vector<sq::LaunchTable> tables;   // grouped kernel: one CTA per item
    std::vector<int> grids;
    int smem_bytes = 0, qmax = 0;
    unsigned mode = 0;
    // cluster kernel (channels wider than one CTA): one launch per layer
    struct Wide { LayerDesc d; int cluster, kpc, smem; };
    std::vector<Wide> wide;
    // pipelined kernel (layers of long 3x3 channels): one item per output channel
    std::vector<sq::LaunchTable> pipe_tables;
    std::vector<int> pipe_items, pipe_set_stride, pipe_slot;
    std::vector<int> pipe_stream;   // 1: the launch goes to the streaming kernel (plain int8 output); pipe_set_stride then
    std::vector<int> pipe_nmax;     // holds the longest channel in weights and pipe_nmax the same in kernels
    // Scratch of the streaming kernel's launches (what SQuant-C needs of every kernel one step later: four
    // sets of 18 KB per thread block), allocated at the plan's first launch, freed with the plan.
    mutable std::vector<void *> pipe_scratch;
    ParamPlan() = default;
    ParamPlan(ParamPlan &&) = default;
    ParamPlan &operator=(ParamPlan &&) = default;
    ParamPlan(const ParamPlan &) = delete;
    ParamPlan &operator=(const ParamPlan &) = delete;
    ~ParamPlan()
    {
        for (void *q : pipe_scratch)
            if (q) cudaFree(q);
    }
    mutable bool slots_clean = false;   // the work counters of pipe_slot have been zeroed on the stream of the plan's first launch
};

int g_next_slot = 0;   // next work-counter slot of the pipelined kernel; guarded by g_mutex

// Layers the pipelined kernel takes: 3x3, more than 8192 weights per output channel (the grouped
// kernel gives such a channel a whole CTA), input channels a multiple of four, SQuant-K on, absmax
// scales, and two buffer sets fit the shared memory of one SM.
bool pipe_eligible(const squant_layer &l, const LayerDesc &d, const squant_options &o, int max_smem)
{
    if (d.K != 9 || (d.N & 3) != 0 || d.NK <= 8192) return false;
    if (!(o.mode & SQUANT_MODE_K) || l.scales_in) return false;
    if ((reinterpret_cast<uintptr_t>(l.w) & 15) || (reinterpret_cast<uintptr_t>(l.codes) & 15)) return false;
    return 2 * d.slice_bytes + sq::kPipeCtrlBytes <= max_smem;
}

// Of those, the streaming kernel takes the layers with plain int8 codes and nothing else to emit.
bool stream_eligible(const squant_layer &l, const LayerDesc &d, const squant_options &o, int max_smem)
{
    if (l.dequant || l.dequant_bf16 || (o.flags & SQUANT_FLAG_PACK_INT4)) return false;
    if (d.N > 4 * sq::kStreamQuantThreads) return false;   // one quad of kernels per quantizer thread
    return sq::stream_layout(d.NK, d.N).total <= max_smem;
}

int build_param_plan(const squant_layer *layers, int32_t n_layers, const squant_options &o,
                     int max_smem, ParamPlan &p)
{
    p.qmax = (1 << (o.bits - 1)) - 1;
    p.mode = o.mode | ((o.flags & SQUANT_FLAG_PACK_INT4) ? sq::kModePackInt4 : 0u) |
             ((o.flags & SQUANT_FLAG_NARROW_RANGE) ? 0u : sq::kModeWideRange);
    p.smem_bytes = 0;
    std::vector<LayerDesc> descs(n_layers);
    std::vector<int> order, piped, streamed;
    for (int i = 0; i < n_layers; ++i) {
        const int64_t cta_smem = layout_layer(layers[i], descs[i], o.mode, o.flags);
        if (cta_smem > max_smem || descs[i].NK > kMaxChannelElems) {
            // a cluster of 2, 4 or 8 CTAs per output channel, each with an even number of kernels
            if ((o.mode & SQUANT_MODE_C) && !(o.mode & SQUANT_MODE_K) && descs[i].K > 1) return SQUANT_ERR_TOO_WIDE;   // E|C selects among elements: one CTA only
            ParamPlan::Wide w{descs[i], 0, 0, 0};
            for (int c = 2; c <= sq::kWideMaxCluster && !w.cluster; c *= 2) {
                const int kpc = (((descs[i].N + c - 1) / c) + 1) & ~1;
                const sq::WideLayout wl = sq::wide_layout(kpc, descs[i].K);
                if (wl.total <= max_smem) { w.cluster = c; w.kpc = kpc; w.smem = wl.total; }
            }
            if (!w.cluster) return SQUANT_ERR_TOO_WIDE;
            p.wide.push_back(w);
            continue;
        }
        if (pipe_eligible(layers[i], descs[i], o, max_smem)) {
            (stream_eligible(layers[i], descs[i], o, max_smem) ? streamed : piped).push_back(i);
            continue;
        }
        if (cta_smem > p.smem_bytes) p.smem_bytes = static_cast<int>(cta_smem);
        order.push_back(i);
    }
    for (int kind = 0; kind < 2; ++kind) {
    const std::vector<int> &piped_k = kind ? streamed : piped;
    for (size_t base = 0; base < piped_k.size(); base += sq::kMaxParamLayers) {
        const int n = static_cast<int>(std::min<size_t>(piped_k.size() - base, sq::kMaxParamLayers));
        p.pipe_tables.emplace_back();
        sq::LaunchTable &t = p.pipe_tables.back();
        std::memset(&t, 0, sizeof(t));
        t.n_layers = n;
        for (int st = 1; st < n; st <<= 1) t.top_step = st;
        int items = 0, stride = 0;
        for (int j = 0; j < n; ++j) {
            const LayerDesc &d = descs[piped_k[base + j]];
            t.layers[j] = d;
            t.first_item[j] = items;
            items += d.M;
            stride = std::max(stride, d.slice_bytes);
        }
        for (int j = n; j <= sq::kMaxParamLayers; ++j) t.first_item[j] = items;
        // One layout for every layer of the launch, that of the widest one: the staging area of a
        // long channel must not reach into the buffers the finishers still use for a shorter one
        // that had the set before, and the channel-step scratch is found (and cleared) without
        // knowing the layer.  It sits at the end of a set.
        int widest = 0;
        for (int j = 1; j < n; ++j)
            if (t.layers[j].slice_bytes > t.layers[widest].slice_bytes) widest = j;
        for (int j = 0; j < n; ++j) {
            LayerDesc &d = t.layers[j];
            const LayerDesc &wd = t.layers[widest];
            d.off_codes = wd.off_codes; d.off_ev = wd.off_ev; d.off_vv = wd.off_vv; d.off_vi = wd.off_vi;
            d.off_hist = wd.off_hist; d.off_red = wd.off_red; d.slice_bytes = wd.slice_bytes;
        }
        int nk_max = 0, n_max = 0;
        for (int j = 0; j < n; ++j) {
            nk_max = std::max(nk_max, t.layers[j].NK);
            n_max = std::max(n_max, t.layers[j].N);
        }
        p.pipe_items.push_back(items);
        p.pipe_set_stride.push_back(kind ? nk_max : stride);
        p.pipe_stream.push_back(kind);
        p.pipe_scratch.push_back(nullptr);
        p.pipe_nmax.push_back(n_max);
        p.pipe_slot.push_back(g_next_slot);
        g_next_slot = (g_next_slot + 1) % sq::kTicketSlots;
    }
    }
    n_layers = static_cast<int32_t>(order.size());   // the grouped kernel takes the rest
    // Estimated duration of one CTA of the layer.  Kernel sizes other than 1x1 and 3x3 take the
    // general per-thread path, which is latency-bound and far slower per weight (a 7x7 stem CTA
    // is the longest of a whole ResNet), so those start first.
    auto cta_work = [&](int i) {
        const LayerDesc &d = descs[i];
        const int64_t groups = sq::kCtaThreads / d.g;
        const int64_t per_channel = (d.K == 1 || d.K == 9) ? d.NK : static_cast<int64_t>(d.NK) * 64 * d.K;
        return (groups < d.M ? groups : d.M) * per_channel;
    };
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return cta_work(a) > cta_work(b); });
    for (int base = 0; base < n_layers; base += sq::kMaxParamLayers) {
        const int n = (n_layers - base < sq::kMaxParamLayers) ? n_layers - base : sq::kMaxParamLayers;
        p.tables.emplace_back();
        sq::LaunchTable &t = p.tables.back();
        std::memset(&t, 0, sizeof(t));
        t.n_layers = n;
        t.top_step = 0;
        for (int st = 1; st < n; st <<= 1) t.top_step = st;
        int items = 0;
        for (int j = 0; j < n; ++j) {
            const LayerDesc &d = descs[order[base + j]];
            const int groups = sq::kCtaThreads / d.g;
            t.layers[j] = d;
            t.first_item[j] = items;
            items += (d.M + groups - 1) / groups;
        }
        for (int j = n; j <= sq::kMaxParamLayers; ++j) t.first_item[j] = items;
        p.grids.push_back(items);
    }
    return SQUANT_OK;
}

// Launch tables are plain host data; the most recent ones are kept, keyed by the exact
// descriptors and options, so that a repeated call only enqueues its kernel(s).
struct CachedPlan {
    int device = -1;
    std::string key;
    ParamPlan plan;
};

std::list<CachedPlan> g_plans;              // most recently used first
std::vector<int> g_smem_limit_by_device;   // opt-in limit set on the kernels, per device
std::vector<int> g_sm_count_by_device;     // multiprocessors, per device

std::string plan_key(const squant_layer *layers, int32_t n_layers, const squant_options &o)
{
    std::string k(reinterpret_cast<const char *>(&o), sizeof(o));
    k.append(reinterpret_cast<const char *>(layers), sizeof(squant_layer) * static_cast<size_t>(n_layers));
    return k;
}

int device_smem_limit(int device, int &limit)
{
    if (static_cast<int>(g_smem_limit_by_device.size()) <= device)
        g_smem_limit_by_device.resize(device + 1, 0);
    if (g_smem_limit_by_device[device] == 0) {
        int v = 0;
        SQ_CUDA(cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, device));
        SQ_CUDA(cudaFuncSetAttribute(sq::squant_model_kernel,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, v));
        SQ_CUDA(cudaFuncSetAttribute(sq::squant_table_kernel,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, v));
        SQ_CUDA(cudaFuncSetAttribute(sq::squant_pipe_kernel,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, v));
        SQ_CUDA(cudaFuncSetAttribute(sq::squant_wide_kernel,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, v));
        SQ_CUDA(cudaFuncSetAttribute(sq::squant_stream_kernel,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, v));
        int sms = 0;
        SQ_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
        if (static_cast<int>(g_sm_count_by_device.size()) <= device) g_sm_count_by_device.resize(device + 1, 0);
        g_sm_count_by_device[device] = sms;
        g_smem_limit_by_device[device] = v;
    }
    limit = g_smem_limit_by_device[device];
    return SQUANT_OK;
}

int get_plan(const squant_layer *layers, int32_t n_layers, const squant_options &o, const ParamPlan *&out)
{
    int device = 0;
    SQ_CUDA(cudaGetDevice(&device));
    std::string key = plan_key(layers, n_layers, o);
    for (auto it = g_plans.begin(); it != g_plans.end(); ++it) {
        if (it->device == device && it->key == key) {
            g_plans.splice(g_plans.begin(), g_plans, it);
            out = &g_plans.front().plan;
            return SQUANT_OK;
        }
    }
    int limit = 0;
    int rc = device_smem_limit(device, limit);
    if (rc) return rc;
    CachedPlan cp;
    cp.device = device;
    cp.key = std::move(key);
    rc = build_param_plan(layers, n_layers, o, limit, cp.plan);
    if (rc) return rc;
    if (g_plans.size() >= kMaxPlans) g_plans.pop_back();
    g_plans.push_front(std::move(cp));
    out = &g_plans.front().plan;
    return SQUANT_OK;
}

// Device address of a work counter (done = false) or of its "CTAs finished" twin (done = true).
void *ticket_address(int slot, bool done)
{
    static std::vector<std::pair<unsigned *, unsigned *>> base;   // per device; guarded by g_mutex
    int device = 0;
    cudaGetDevice(&device);
    if (static_cast<int>(base.size()) <= device) base.resize(device + 1, {nullptr, nullptr});
    if (!base[device].first) {
        cudaGetSymbolAddress(reinterpret_cast<void **>(&base[device].first), sq::g_ticket);
        cudaGetSymbolAddress(reinterpret_cast<void **>(&base[device].second), sq::g_done);
    }
    return (done ? base[device].second : base[device].first) + slot;
}

int launch_plan(const ParamPlan &p, cudaStream_t stream)
{
    // A work-counter slot comes to a plan in an unknown state (a plan that was evicted, or a launch
    // that failed, may have left it dirty): zero it in stream order before the plan's first launch.
    if (!p.slots_clean) {
        for (size_t c = 0; c < p.pipe_tables.size(); ++c) {
            SQ_CUDA(cudaMemsetAsync(ticket_address(p.pipe_slot[c], false), 0, sizeof(unsigned), stream));
            SQ_CUDA(cudaMemsetAsync(ticket_address(p.pipe_slot[c], true), 0, sizeof(unsigned), stream));
        }
        p.slots_clean = true;
    }
    // long 3x3 channels first: one persistent CTA per multiprocessor
    for (size_t c = 0; c < p.pipe_tables.size(); ++c) {
        if (p.pipe_items[c] == 0) continue;
        int device = 0;
        SQ_CUDA(cudaGetDevice(&device));
        const int grid = std::min(p.pipe_items[c], std::max(g_sm_count_by_device[device], 1));
        if (p.pipe_stream[c]) {
            const int smem = sq::stream_layout(p.pipe_set_stride[c], p.pipe_nmax[c]).total;
            if (!p.pipe_scratch[c]) {
                const size_t bytes = static_cast<size_t>(std::max(g_sm_count_by_device[device], 1)) * sq::kStreamHeldSets * sq::kStreamHeldBytes;
                if (cudaMalloc(&p.pipe_scratch[c], bytes) != cudaSuccess) {
                    cudaGetLastError();   // the failed allocation is reported by the return code, not left pending
                    p.pipe_scratch[c] = nullptr;
                    return SQUANT_ERR_NOMEM;
                }
            }
            sq::squant_stream_kernel<<<grid, sq::kStreamThreads, smem, stream>>>(p.pipe_tables[c], p.qmax, p.mode, p.pipe_items[c],
                                                                             p.pipe_slot[c], p.pipe_set_stride[c], p.pipe_nmax[c],
                                                                             static_cast<unsigned char *>(p.pipe_scratch[c]));
        } else {
            const int smem = 2 * p.pipe_set_stride[c] + sq::kPipeCtrlBytes;
            sq::squant_pipe_kernel<<<grid, sq::kPipeThreads, smem, stream>>>(p.pipe_tables[c], p.qmax, p.mode, p.pipe_items[c],
                                                                         p.pipe_slot[c], p.pipe_set_stride[c]);
        }
        SQ_CUDA(cudaGetLastError());
        g_launches.fetch_add(1, std::memory_order_relaxed);
    }
    for (size_t c = 0; c < p.tables.size(); ++c) {
        if (p.grids[c] == 0) continue;
        sq::squant_model_kernel<<<p.grids[c], sq::kCtaThreads, p.smem_bytes, stream>>>(p.tables[c], p.qmax, p.mode);
        SQ_CUDA(cudaGetLastError());
        g_launches.fetch_add(1, std::memory_order_relaxed);
    }
    for (const ParamPlan::Wide &w : p.wide) {   // one cluster per output channel
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(w.d.M) * w.cluster);
        cfg.blockDim = dim3(sq::kWideThreads);
        cfg.dynamicSmemBytes = static_cast<size_t>(w.smem);
        cfg.stream = stream;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = static_cast<unsigned>(w.cluster);
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        SQ_CUDA(cudaLaunchKernelEx(&cfg, sq::squant_wide_kernel, w.d, p.qmax, p.mode, w.kpc));
        g_launches.fetch_add(1, std::memory_order_relaxed);
    }
    return SQUANT_OK;
}

// Device staging of the host-buffer entry point, one arena per device, grown on demand.
struct Arena { void *ptr = nullptr; size_t bytes = 0; };
std::vector<Arena> g_arenas;

// Copy streams and events of the host-buffer entry point, one set per device, created on first
// use: uploads, kernels and downloads of consecutive chunks of layers overlap.
struct HostPipe {
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr;
    std::vector<cudaEvent_t> uploaded, computed;
};
std::vector<HostPipe> g_host_pipes;
constexpr size_t kHostChunkBytes = 64u << 20;   // weights per chunk: large enough to hide the launches

int host_pipe(int device, size_t chunks, HostPipe *&out)
{
    if (static_cast<int>(g_host_pipes.size()) <= device) g_host_pipes.resize(device + 1);
    HostPipe &hp = g_host_pipes[device];
    if (!hp.in) {
        SQ_CUDA(cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking));
        SQ_CUDA(cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking));
        SQ_CUDA(cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming));
    }
    while (hp.uploaded.size() < chunks) {
        cudaEvent_t a = nullptr, b = nullptr;
        SQ_CUDA(cudaEventCreateWithFlags(&a, cudaEventDisableTiming));
        SQ_CUDA(cudaEventCreateWithFlags(&b, cudaEventDisableTiming));
        hp.uploaded.push_back(a);
        hp.computed.push_back(b);
    }
    out = &hp;
    return SQUANT_OK;
}

inline size_t align256(size_t v) { return (v + 255) & ~static_cast<size_t>(255); }

// ---- launch table of squant_quantize_layer_noalloc: part of the library image, never allocated.
// Layout: one LayerDesc in the first 256 bytes, then up to SQUANT_NOALLOC_MAX_CTAS Items.
// In host code the name below is only a handle of the symbol; the address a kernel can use comes
// from cudaGetSymbolAddress, taken once per device with that device current.
static_assert(sizeof(LayerDesc) <= 256, "layer descriptor must fit the table header");
static_assert(sizeof(Item) == 8, "table size in squant.h assumes 8-byte entries");
static __device__ __align__(256) unsigned char g_noalloc_table[SQUANT_NOALLOC_TABLE_BYTES];
unsigned char g_noalloc_host[SQUANT_NOALLOC_TABLE_BYTES];   // host image, guarded by g_mutex
std::vector<void *> g_noalloc_dev;                          // per device: address of the table

int noalloc_table_address(int device, void *&ptr)
{
    if (static_cast<int>(g_noalloc_dev.size()) <= device) g_noalloc_dev.resize(device + 1, nullptr);
    if (!g_noalloc_dev[device]) {
        void *p = nullptr;
        SQ_CUDA(cudaGetSymbolAddress(&p, g_noalloc_table));   // current device is `device`
        g_noalloc_dev[device] = p;
    }
    ptr = g_noalloc_dev[device];
    return SQUANT_OK;
}

}  // namespace

extern "C" {

int squant_quantize_model(const squant_layer *layers, int32_t n_layers, const squant_options *opt,
                          void *cuda_stream)
{
    squant_options o;
    int rc = validate(layers, n_layers, opt, true, o);
    if (rc) return rc;
    if (n_layers == 0) return SQUANT_OK;
    std::lock_guard<std::mutex> lock(g_mutex);
    const ParamPlan *pp = nullptr;
    rc = get_plan(layers, n_layers, o, pp);
    if (rc) return rc;
    return launch_plan(*pp, static_cast<cudaStream_t>(cuda_stream));
}

int squant_quantize_layer(const squant_layer *layer, const squant_options *opt, void *cuda_stream)
{
    if (!layer) return SQUANT_ERR_NULL;
    return squant_quantize_model(layer, 1, opt, cuda_stream);
}

int squant_quantize_model_host(const squant_layer *layers, int32_t n_layers,
                               const squant_options *opt, void *cuda_stream)
{
    squant_options o;
    int rc = validate(layers, n_layers, opt, true, o);
    if (rc) return rc;
    if (n_layers == 0) return SQUANT_OK;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    std::lock_guard<std::mutex> lock(g_mutex);
    int device = 0;
    SQ_CUDA(cudaGetDevice(&device));
    // carve one device arena: per layer weights, codes, scales, kernel sums, channel sums
    std::vector<squant_layer> dev(layers, layers + n_layers);
    std::vector<size_t> off(static_cast<size_t>(n_layers) * 8);
    size_t total = 0;
    for (int i = 0; i < n_layers; ++i) {
        const squant_layer &l = layers[i];
        const size_t n = static_cast<size_t>(l.cin) * l.kh * l.kw * l.cout;
        off[8 * i + 0] = total; total += align256(n * 4);
        const size_t code_bytes = (o.flags & SQUANT_FLAG_PACK_INT4)
                                      ? static_cast<size_t>(l.cout) * ((static_cast<size_t>(l.cin) * l.kh * l.kw + 1) / 2) : n;
        off[8 * i + 1] = total; total += align256(code_bytes);
        off[8 * i + 2] = total; total += align256(static_cast<size_t>(l.cout) * 4);
        off[8 * i + 3] = total; total += l.kernel_err ? align256(static_cast<size_t>(l.cout) * l.cin * 4) : 0;
        off[8 * i + 4] = total; total += l.channel_err ? align256(static_cast<size_t>(l.cout) * 4) : 0;
        off[8 * i + 5] = total; total += l.dequant ? align256(n * 4) : 0;
        off[8 * i + 6] = total; total += l.scales_in ? align256(static_cast<size_t>(l.cout) * 4) : 0;
        off[8 * i + 7] = total; total += l.dequant_bf16 ? align256(n * 2) : 0;
    }
    if (static_cast<int>(g_arenas.size()) <= device) g_arenas.resize(device + 1);
    Arena &a = g_arenas[device];
    if (a.bytes < total) {
        if (a.ptr) { SQ_CUDA(cudaDeviceSynchronize()); SQ_CUDA(cudaFree(a.ptr)); a.ptr = nullptr; a.bytes = 0; }
        cudaError_t e = cudaMalloc(&a.ptr, total);
        if (e != cudaSuccess) { a.ptr = nullptr; return e == cudaErrorMemoryAllocation ? SQUANT_ERR_NOMEM : cuda_fail(e, "cudaMalloc"); }
        a.bytes = total;
    }
    unsigned char *base = static_cast<unsigned char *>(a.ptr);
    for (int i = 0; i < n_layers; ++i) {
        const squant_layer &l = layers[i];
        dev[i].w = reinterpret_cast<const float *>(base + off[8 * i + 0]);
        dev[i].codes = reinterpret_cast<int8_t *>(base + off[8 * i + 1]);
        dev[i].scales = reinterpret_cast<float *>(base + off[8 * i + 2]);
        dev[i].kernel_err = l.kernel_err ? reinterpret_cast<float *>(base + off[8 * i + 3]) : nullptr;
        dev[i].channel_err = l.channel_err ? reinterpret_cast<float *>(base + off[8 * i + 4]) : nullptr;
        dev[i].dequant = l.dequant ? reinterpret_cast<float *>(base + off[8 * i + 5]) : nullptr;
        dev[i].scales_in = l.scales_in ? reinterpret_cast<const float *>(base + off[8 * i + 6]) : nullptr;
        dev[i].dequant_bf16 = l.dequant_bf16 ? reinterpret_cast<uint16_t *>(base + off[8 * i + 7]) : nullptr;
    }
    // Chunks of consecutive layers (about kHostChunkBytes of weights each).  Uploads run on one
    // copy stream, each chunk's launches on the caller's stream once its upload is done, its
    // downloads on a second copy stream once its launches are done: the two copy directions and
    // the kernels overlap.
    std::vector<int> chunk_first(1, 0);
    {
        size_t acc = 0;
        for (int i = 0; i < n_layers; ++i) {
            acc += static_cast<size_t>(layers[i].cin) * layers[i].kh * layers[i].kw * layers[i].cout * 4;
            if (acc >= kHostChunkBytes && i + 1 < n_layers) { chunk_first.push_back(i + 1); acc = 0; }
        }
        chunk_first.push_back(n_layers);
    }
    const size_t chunks = chunk_first.size() - 1;
    HostPipe *hp = nullptr;
    rc = host_pipe(device, chunks, hp);
    if (rc) return rc;
    SQ_CUDA(cudaEventRecord(hp->start, stream));          // uploads follow what the caller's stream holds so far
    SQ_CUDA(cudaStreamWaitEvent(hp->in, hp->start, 0));
    for (size_t c = 0; c < chunks; ++c) {
        for (int i = chunk_first[c]; i < chunk_first[c + 1]; ++i) {
            const squant_layer &l = layers[i];
            const size_t n = static_cast<size_t>(l.cin) * l.kh * l.kw * l.cout;
            SQ_CUDA(cudaMemcpyAsync(base + off[8 * i + 0], l.w, n * 4, cudaMemcpyHostToDevice, hp->in));
            if (l.scales_in)
                SQ_CUDA(cudaMemcpyAsync(base + off[8 * i + 6], l.scales_in, static_cast<size_t>(l.cout) * 4, cudaMemcpyHostToDevice, hp->in));
        }
        SQ_CUDA(cudaEventRecord(hp->uploaded[c], hp->in));
    }
    for (size_t c = 0; c < chunks; ++c) {
        const int first = chunk_first[c], count = chunk_first[c + 1] - first;
        SQ_CUDA(cudaStreamWaitEvent(stream, hp->uploaded[c], 0));
        const ParamPlan *pp = nullptr;
        rc = get_plan(dev.data() + first, count, o, pp);
        if (rc) return rc;
        rc = launch_plan(*pp, stream);
        if (rc) return rc;
        SQ_CUDA(cudaEventRecord(hp->computed[c], stream));
        SQ_CUDA(cudaStreamWaitEvent(hp->out, hp->computed[c], 0));
        for (int i = first; i < first + count; ++i) {
            const squant_layer &l = layers[i];
            const size_t n = static_cast<size_t>(l.cin) * l.kh * l.kw * l.cout;
            const size_t code_bytes = (o.flags & SQUANT_FLAG_PACK_INT4)
                                          ? static_cast<size_t>(l.cout) * ((static_cast<size_t>(l.cin) * l.kh * l.kw + 1) / 2) : n;
            SQ_CUDA(cudaMemcpyAsync(l.codes, dev[i].codes, code_bytes, cudaMemcpyDeviceToHost, hp->out));
            SQ_CUDA(cudaMemcpyAsync(l.scales, dev[i].scales, static_cast<size_t>(l.cout) * 4, cudaMemcpyDeviceToHost, hp->out));
            if (l.kernel_err)
                SQ_CUDA(cudaMemcpyAsync(l.kernel_err, dev[i].kernel_err, static_cast<size_t>(l.cout) * l.cin * 4, cudaMemcpyDeviceToHost, hp->out));
            if (l.channel_err)
                SQ_CUDA(cudaMemcpyAsync(l.channel_err, dev[i].channel_err, static_cast<size_t>(l.cout) * 4, cudaMemcpyDeviceToHost, hp->out));
            if (l.dequant)
                SQ_CUDA(cudaMemcpyAsync(l.dequant, dev[i].dequant, n * 4, cudaMemcpyDeviceToHost, hp->out));
            if (l.dequant_bf16)
                SQ_CUDA(cudaMemcpyAsync(l.dequant_bf16, dev[i].dequant_bf16, n * 2, cudaMemcpyDeviceToHost, hp->out));
        }
    }
    SQ_CUDA(cudaStreamSynchronize(hp->out));
    SQ_CUDA(cudaStreamSynchronize(stream));
    return SQUANT_OK;
}

int squant_quantize_layer_noalloc(const squant_layer *layer, const squant_options *opt,
                                  void *cuda_stream)
{
    if (!layer) return SQUANT_ERR_NULL;
    squant_options o;
    int rc = validate(layer, 1, opt, true, o);
    if (rc) return rc;
    HostPlan hp;   // host-side bookkeeping only; nothing below allocates device memory
    rc = build_plan(layer, 1, o, kMaxSmemFallback, hp);
    if (rc) return rc;
    if (hp.items.size() > static_cast<size_t>(SQUANT_NOALLOC_MAX_CTAS)) return SQUANT_ERR_LIMIT;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    std::lock_guard<std::mutex> lock(g_mutex);
    {   // the table upload below reads a host image that the next call rewrites: not for a captured stream
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        SQ_CUDA(cudaStreamIsCapturing(stream, &cap));
        if (cap != cudaStreamCaptureStatusNone) return SQUANT_ERR_CAPTURE;
    }
    int device = 0;
    SQ_CUDA(cudaGetDevice(&device));
    int limit = 0;
    rc = device_smem_limit(device, limit);
    if (rc) return rc;
    if (hp.smem_bytes > limit) return SQUANT_ERR_TOO_WIDE;
    void *table = nullptr;
    rc = noalloc_table_address(device, table);
    if (rc) return rc;
    const size_t ibytes = sizeof(Item) * hp.items.size();
    std::memcpy(g_noalloc_host, hp.layers.data(), sizeof(LayerDesc));
    std::memcpy(g_noalloc_host + 256, hp.items.data(), ibytes);
    // Pageable source: the runtime has taken its copy of the bytes when this returns, so the host
    // image may be rewritten by the next call; the device-side copy is ordered on `stream`.
    SQ_CUDA(cudaMemcpyAsync(table, g_noalloc_host, 256 + ibytes, cudaMemcpyHostToDevice, stream));
    const LayerDesc *dl = static_cast<const LayerDesc *>(table);
    const Item *di = reinterpret_cast<const Item *>(static_cast<const unsigned char *>(table) + 256);
    sq::squant_table_kernel<<<static_cast<unsigned>(hp.items.size()), sq::kCtaThreads, hp.smem_bytes, stream>>>(
        dl, di, hp.qmax, hp.mode);
    SQ_CUDA(cudaGetLastError());
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return SQUANT_OK;
}

int squant_plan_info(const squant_layer *layers, int32_t n_layers, const squant_options *opt,
                     int32_t *grid_ctas, int32_t *cta_threads, int32_t *dynamic_smem_bytes)
{
    squant_options o;
    int rc = validate(layers, n_layers, opt, false, o);
    if (rc) return rc;
    HostPlan hp;
    rc = build_plan(layers, n_layers, o, kMaxSmemFallback, hp);
    if (rc) return rc;
    if (grid_ctas) *grid_ctas = static_cast<int32_t>(hp.items.size());
    if (cta_threads) *cta_threads = sq::kCtaThreads;
    if (dynamic_smem_bytes) *dynamic_smem_bytes = hp.smem_bytes;
    return SQUANT_OK;
}

int squant_selfcheck_division(const float *scales, int32_t n, int32_t bits, uint64_t *mismatches,
                              void *cuda_stream)
{
    if (!scales || !mismatches) return SQUANT_ERR_NULL;
    if (n <= 0 || n > 65535) return SQUANT_ERR_SHAPE;
    if (bits < 2 || bits > 8) return SQUANT_ERR_BITS;
    for (int i = 0; i < n; ++i)
        if (!(scales[i] >= 0x1p-60f && scales[i] <= 0x1p60f)) return SQUANT_ERR_SHAPE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    float *d_s = nullptr;
    unsigned long long *d_m = nullptr;
    SQ_CUDA(cudaMalloc(&d_s, sizeof(float) * n));
    cudaError_t e = cudaMalloc(&d_m, sizeof(unsigned long long) * n);
    if (e != cudaSuccess) { cudaFree(d_s); return cuda_fail(e, "cudaMalloc"); }
    e = cudaMemcpyAsync(d_s, scales, sizeof(float) * n, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(d_m, 0, sizeof(unsigned long long) * n, stream);
    if (e == cudaSuccess) {
        sq::selfcheck_division_kernel<<<dim3(1184, n), 256, 0, stream>>>(d_s, n, (1 << (bits - 1)) - 1, d_m);
        e = cudaGetLastError();
        g_launches.fetch_add(1, std::memory_order_relaxed);
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(mismatches, d_m, sizeof(unsigned long long) * n, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    cudaFree(d_s);
    cudaFree(d_m);
    if (e != cudaSuccess) return cuda_fail(e, "squant_selfcheck_division");
    return SQUANT_OK;
}

int squant_device_status(void)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    SQ_CUDA(cudaDeviceSynchronize());
    int st = 0;
    SQ_CUDA(cudaMemcpyFromSymbol(&st, sq::g_device_status, sizeof(int)));
    if (st == 0) return SQUANT_OK;
    const int zero = 0;
    SQ_CUDA(cudaMemcpyToSymbol(sq::g_device_status, &zero, sizeof(int)));
    // a launch that gave up may have left its work counter half drawn: all plans start clean again
    SQ_CUDA(cudaMemset(ticket_address(0, false), 0, sizeof(unsigned) * sq::kTicketSlots));
    SQ_CUDA(cudaMemset(ticket_address(0, true), 0, sizeof(unsigned) * sq::kTicketSlots));
    return SQUANT_ERR_TIMEOUT;
}

int squant_debug_violations(int32_t *count, int32_t *first_site)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    SQ_CUDA(cudaDeviceSynchronize());
    unsigned n = 0;
    int site = 0;
    SQ_CUDA(cudaMemcpyFromSymbol(&n, sq::g_debug_violations, sizeof(n)));
    SQ_CUDA(cudaMemcpyFromSymbol(&site, sq::g_debug_site, sizeof(site)));
    if (count) *count = static_cast<int32_t>(n);
    if (first_site) *first_site = site;
    const unsigned zero = 0;
    SQ_CUDA(cudaMemcpyToSymbol(sq::g_debug_violations, &zero, sizeof(zero)));
    SQ_CUDA(cudaMemcpyToSymbol(sq::g_debug_site, &zero, sizeof(int)));
#ifdef SQUANT_DEBUG_BOUNDS
    return 1;   // this library was built with the checks
#else
    return SQUANT_OK;
#endif
}

int squant_debug_set_status(int value)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    SQ_CUDA(cudaMemcpyToSymbol(sq::g_device_status, &value, sizeof(int)));
    return SQUANT_OK;
}

int squant_debug_wait_expires(int32_t max_polls, void *cuda_stream)
{
    if (max_polls < 1 || max_polls > 4096) return SQUANT_ERR_SHAPE;
    sq::debug_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(max_polls);
    SQ_CUDA(cudaGetLastError());
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return SQUANT_OK;
}

int64_t squant_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char *squant_strerror(int code)
{
    switch (code) {
        case SQUANT_OK: return "success";
        case SQUANT_ERR_NULL: return "a required pointer is NULL";
        case SQUANT_ERR_SHAPE: return "a layer dimension is not positive or the element count overflows";
        case SQUANT_ERR_BITS: return "bits must be in 2..8 (2..4 with SQUANT_FLAG_PACK_INT4)";
        case SQUANT_ERR_MODE: return "mode mask must contain E (E, E|K, E|C or E|K|C); unknown mode or flag bits are rejected";
        case SQUANT_ERR_ALIGN: return "float pointers must be 4-byte aligned";
        case SQUANT_ERR_TOO_WIDE: return "an output channel (cin*kh*kw) does not fit the on-chip path, not even spread over a cluster of 8 thread blocks";
        case SQUANT_ERR_CUDA: return "a CUDA runtime call failed (see squant_last_cuda_error)";
        case SQUANT_ERR_NOMEM: return "out of host or device memory";
        case SQUANT_ERR_TIMEOUT: return "a kernel gave up a bounded wait on an asynchronous copy; outputs of that launch are incomplete";
        case SQUANT_ERR_CAPTURE: return "squant_quantize_layer_noalloc was called on a stream that is being captured; it uploads its launch table from a host image that the next call rewrites";
        case SQUANT_ERR_LIMIT: return "the layer needs more thread blocks than the fixed launch table of squant_quantize_layer_noalloc holds (SQUANT_NOALLOC_MAX_CTAS); split it by output-channel range";
        default: return "unknown squant error code";
    }
}

const char *squant_last_cuda_error(void) { return t_cuda_error.c_str(); }

int squant_shutdown(void)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    int cur = 0;
    const bool have = cudaGetDevice(&cur) == cudaSuccess;
    g_plans.clear();
    for (size_t d = 0; d < g_arenas.size(); ++d) {
        if (g_arenas[d].ptr) { cudaSetDevice(static_cast<int>(d)); cudaDeviceSynchronize(); cudaFree(g_arenas[d].ptr); }
    }
    g_arenas.clear();
    for (size_t d = 0; d < g_host_pipes.size(); ++d) {
        HostPipe &hp = g_host_pipes[d];
        if (!hp.in) continue;
        cudaSetDevice(static_cast<int>(d));
        for (cudaEvent_t e : hp.uploaded) cudaEventDestroy(e);
        for (cudaEvent_t e : hp.computed) cudaEventDestroy(e);
        cudaEventDestroy(hp.start);
        cudaStreamDestroy(hp.in);
        cudaStreamDestroy(hp.out);
    }
    g_host_pipes.clear();
    if (have) cudaSetDevice(cur);
    return SQUANT_OK;
}

}  // extern "C"
