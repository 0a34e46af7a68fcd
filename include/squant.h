/*
 * squant.h - C ABI of the B200 (sm_100a) SQuant weight quantizer.
 *
 * The library turns the fp32 weights of convolution / fully connected layers into low-bit
 * integer codes with the progressive solver of the SQuant paper (arXiv 2202.07471,
 * Algorithm 1 "Progressive SQuant Algorithm"):
 *
 *   scale     per output channel, symmetric:  s_m = max|W[m]| / qmax,  qmax = 2^(bits-1) - 1
 *             (the paper takes s as an input of Algorithm 1 and sets the range per output
 *             channel, Sec. 4; a channel with max|W| < 2^-100 gets s_m = 1 and all-zero codes)
 *   SQuant-E  Eq. 9 / Algorithm 1 "Scale and SQuant-E": x = w / s_m in IEEE fp32, round to
 *             nearest (ties to even); perturbation p = code - x, held as the integer
 *             nearbyint(p * 2^30) from here on, so that all sums are exact
 *   SQuant-K  Eq. 10 / Algorithm 2 (SQuantFlip) on each kernel W[m][n][:]: with e the sum of the
 *             kernel's perturbations, flip the k = round(|e|) elements that have the sign of
 *             e and the largest |p| by one step, which brings |e| to at most 0.5
 *   update    Algorithm 3 (UpdatePerturbation): each kernel keeps ONE candidate element for
 *             SQuant-C (Over SQuant: the last flipped element, to be flipped back;
 *             Under SQuant: the first un-flipped one)
 *   SQuant-C  Eq. 11 / Algorithm 2 on each output channel: with e_c the sum of ALL perturbations
 *             of the channel, flip the candidates of the k_c = round(|e_c|) kernels whose
 *             candidate has the sign of e_c and the largest |p|, one element per kernel
 *
 * Tie rules: round(|e|) at exactly one half takes the smaller count; equal |p| go to the lower
 * flat index (offset n*K + i inside the output channel).  Results are deterministic and do
 * not depend on launch geometry.
 *
 * Layout: weights and codes are row-major [cout][cin][kh][kw] (a fully connected layer is
 * kh = kw = 1; a depthwise convolution has cin = 1).  One "kernel" is the kh*kw weights
 * W[m][n][:], one "output channel" the cin*kh*kw weights W[m][:][:].
 *
 * Threading: calls may come from several host threads; the library serialises its own
 * bookkeeping.  All work is asynchronous on the given CUDA stream unless stated otherwise.
 */
#ifndef SQUANT_H_
#define SQUANT_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* stages to run (bit mask); SQUANT_MODE_E is mandatory.  E, E|K, E|C and E|K|C are the four
 * variants of the paper's granularity ablation (Table 5); without SQUANT_MODE_K every element
 * is its own candidate for SQuant-C. */
#define SQUANT_MODE_E 1u
#define SQUANT_MODE_K 2u
#define SQUANT_MODE_C 4u
#define SQUANT_MODE_EKC (SQUANT_MODE_E | SQUANT_MODE_K | SQUANT_MODE_C)

/* flags */
#define SQUANT_FLAG_NARROW_RANGE 1u /* codes in [-qmax, qmax] (default); without it the lower
                                       bound is -qmax-1, which the absmax scale never reaches */
#define SQUANT_FLAG_PACK_INT4 2u    /* bits <= 4 only: codes are emitted two per byte (two's
                                       complement nibbles, low nibble = even flat index), every
                                       output channel in a row of ceil(cin*kh*kw / 2) bytes */

/* error codes (0 = success) */
#define SQUANT_OK 0
#define SQUANT_ERR_NULL (-1)        /* a required pointer is NULL */
#define SQUANT_ERR_SHAPE (-2)       /* a dimension is <= 0 or the element count overflows */
#define SQUANT_ERR_BITS (-3)        /* bits outside 2..8 */
#define SQUANT_ERR_MODE (-4)        /* mode mask without SQUANT_MODE_E, or unknown mode / flag bits */
#define SQUANT_ERR_ALIGN (-5)       /* weights / scales / error pointers not 4-byte aligned */
#define SQUANT_ERR_TOO_WIDE (-6)    /* one output channel does not fit the on-chip path */
#define SQUANT_ERR_CUDA (-7)        /* a CUDA runtime call failed; see squant_last_cuda_error() */
#define SQUANT_ERR_NOMEM (-8)       /* host or device allocation failed */
#define SQUANT_ERR_TIMEOUT (-10)    /* a kernel gave up a bounded wait on an asynchronous copy; the
                                       outputs of that launch are incomplete */
#define SQUANT_ERR_CAPTURE (-11)    /* squant_quantize_layer_noalloc on a stream that is being captured */
#define SQUANT_ERR_LIMIT (-9)       /* the layer needs more launch-table entries than the fixed
                                       table of squant_quantize_layer_noalloc holds */

typedef struct squant_options {
    int32_t bits;   /* 2..8; qmax = 2^(bits-1) - 1 */
    uint32_t mode;  /* SQUANT_MODE_* mask; 0 means SQUANT_MODE_EKC */
    uint32_t flags; /* SQUANT_FLAG_* */
} squant_options;

/*
 * One layer.  For squant_quantize_layer / squant_quantize_model every pointer is a DEVICE
 * pointer; for squant_quantize_model_host every pointer is a HOST pointer.  The caller owns
 * all buffers; the library never frees or retains them beyond the call's work on the stream.
 */
typedef struct squant_layer {
    const float *w;      /* in : [cout][cin][kh][kw] fp32, finite values, 4-byte aligned
                                 (16-byte alignment of every channel enables the fast loads) */
    int32_t cout, cin, kh, kw;
    int8_t *codes;       /* out: [cout][cin][kh][kw] int8, or with SQUANT_FLAG_PACK_INT4
                                 [cout][ceil(cin*kh*kw / 2)] bytes of nibble pairs */
    float *scales;       /* out: [cout] */
    float *kernel_err;   /* out, may be NULL: [cout][cin] final signed sum of a kernel's
                                 perturbations, (float)(integer sum) * 2^-30 */
    float *channel_err;  /* out, may be NULL: [cout] final signed sum of a channel's
                                 perturbations */
    float *dequant;      /* out, may be NULL: [cout][cin][kh][kw] fp32 quantized weights
                                 code * s_m - what Algorithm 1 itself returns ("C * s") */
    uint16_t *dequant_bf16; /* out, may be NULL: the same quantized weights as bfloat16 bit patterns
                                 (the fp32 product code * s_m rounded to nearest, ties to even) */
    const float *scales_in; /* in, may be NULL: [cout] caller-supplied scales, the input s of
                                 Algorithm 1.  NULL: absmax scales (above).  With a supplied scale
                                 the clip of Sec. 2.2 really fires: a clipped element keeps its
                                 saturated code, its perturbation enters the kernel and channel
                                 sums, and it is never flipped outward; when fewer candidates exist
                                 than round(|e|) asks for, all are flipped and kernel_err /
                                 channel_err report what is left (then above 0.5).  A scale that
                                 is not a positive finite number is replaced by 1; |w / s| must
                                 stay below 2^12.  `scales` receives the scales used.  Not
                                 available for E|C without K on kernels larger than 1x1
                                 (SQUANT_ERR_MODE). */
} squant_layer;

/*
 * Algorithm 1 on one layer (DEVICE pointers).  Same as squant_quantize_model with one layer.
 */
int squant_quantize_layer(const squant_layer *layer, const squant_options *opt, void *cuda_stream);

/*
 * Algorithm 1 on every layer of a model in one pass (the paper sums per-layer times and notes
 * that layers could be quantized in parallel, Sec. 4.2): ONE grouped kernel launch for all
 * layers, plus one launch of a persistent kernel for those layers whose 3x3 output channels are
 * longer than 8192 weights (cin a multiple of 4 and at most 2048, SQuant-K on, absmax scales): the
 * streaming kernel when only int8 codes are wanted, the pipelined kernel for packed or
 * dequantized outputs.
 *
 *   layers, n_layers  host array of descriptors holding DEVICE pointers; n_layers >= 0
 *   opt               bits / mode / flags shared by all layers; NULL means 4 bit, E|K|C, narrow
 *   cuda_stream       a cudaStream_t (NULL = default stream)
 *
 * The launch table (layer descriptors) travels by value in the kernel's parameter space: the call
 * uploads nothing and never synchronises; more than 96 layers are issued as several launches.
 * Host-side launch tables of recent calls are cached.  The only device memory the call ever
 * allocates is the streaming kernel's scratch area (72 KB per multiprocessor, about 11 MB on a
 * B200): at the FIRST call with given descriptors that has such layers, by cudaMalloc, kept with
 * the cached launch tables and freed with them (so that first call belongs outside any stream
 * capture; callers that cannot allocate at all: see squant_quantize_layer_noalloc).  Outputs are valid when the stream reaches the end of the
 * launches.  The persistent kernels hand out their channels through a counter in device memory
 * that, like the scratch area, belongs to the cached launch tables of these exact descriptors:
 * two calls with the SAME descriptors must not overlap on the GPU (they would race on the
 * outputs anyway); calls with different descriptors may.  All arguments are validated
 * on the host first; a failed call launches nothing and writes nothing.  Returns SQUANT_OK or a
 * negative SQUANT_ERR_* code.
 */
int squant_quantize_model(const squant_layer *layers, int32_t n_layers, const squant_options *opt,
                          void *cuda_stream);

/*
 * The same, with HOST buffers: copies the weights to the current device, runs the launches,
 * copies codes / scales / error sums back and returns when the outputs are in host memory.
 * The layers are taken in chunks of about 64 MB of weights: uploads, launches and downloads of
 * consecutive chunks overlap on two copy streams of the library (created on first use) beside
 * the caller's stream, on which the launches run.  Device staging memory is cached inside the
 * library between calls (cudaMalloc on first use or growth; squant_shutdown frees it).  Pinned
 * host memory gives the copies their full speed and lets them overlap; pageable memory works.
 */
int squant_quantize_model_host(const squant_layer *layers, int32_t n_layers,
                               const squant_options *opt, void *cuda_stream);

/*
 * Geometry of the grouped launch (one thread block per 256/g output channels) that covers
 * these descriptors, as squant_quantize_layer_noalloc issues it (pointers are not dereferenced
 * and may be NULL here).  squant_quantize_model itself sends layers of long 3x3 channels to its
 * pipelined kernel instead, whose grid is one block per multiprocessor.  Any output may be NULL.
 */
int squant_plan_info(const squant_layer *layers, int32_t n_layers, const squant_options *opt,
                     int32_t *grid_ctas, int32_t *cta_threads, int32_t *dynamic_smem_bytes);

/*
 * squant_quantize_layer without any device allocation.  (An addition of this library; the paper
 * has no counterpart.)
 *
 * Who needs it: code that must not call cudaMalloc while it runs - a serving or training process
 * whose framework has handed every free byte of the GPU to its own memory pool (cudaMalloc then
 * fails or fragments the pool), a latency-critical loop that cannot take the device-wide
 * synchronisation cudaMalloc / cudaFree imply, or a host that is only allowed to run
 * pre-loaded code.  This entry point runs the kernel variant that reads its launch table (layer
 * descriptor + one entry per CTA) from global memory, and keeps that table in a fixed array
 * that is part of the library image, so it calls no cudaMalloc, cudaFree or other allocating
 * routine.  Every GPU that loads the library holds that array
 * (SQUANT_NOALLOC_TABLE_BYTES, about 256 KB) until the process exits.
 *
 *   layer, opt, cuda_stream   as for squant_quantize_layer; DEVICE pointers, caller-owned
 *
 * Limits: one layer per call, and the layer's launch must need at most SQUANT_NOALLOC_MAX_CTAS
 * thread blocks (one block handles 256/g output channels, g = 32..256 threads per channel by
 * channel length; squant_plan_info reports the count).  A larger layer is rejected with
 * SQUANT_ERR_LIMIT before anything is launched; split it by output-channel range and call once
 * per part.
 *
 * Sharing: all calls on a device use the same table, and each call overwrites the part it
 * needs (nothing in it has to start at zero; the previous call's entries beyond that part are
 * left behind and never read).  Calls are ordered correctly when they are issued to the same
 * stream.  Two calls whose GPU work can overlap - different streams without an event between
 * them - race: the second call's table upload may land while the first call's kernel is still
 * reading it.  Serialise such calls.
 *
 * The first call on each device looks up the table's device address and raises the kernel's
 * shared-memory limit; make that first call outside any stream capture.  Every call uploads the
 * table from a host image inside the library that the next call rewrites, so a call on a stream
 * that is being captured is refused (SQUANT_ERR_CAPTURE, nothing is enqueued).  The host image is
 * ordinary pageable memory: the runtime stages such an upload through its own buffers, and the call
 * can return only after that, which may mean waiting until earlier work on the stream has let the
 * copy start - a caller in a latency-critical loop should count on the call blocking that long.
 *
 * Results are bit-identical to squant_quantize_layer.  Returns SQUANT_OK or a negative
 * SQUANT_ERR_* code; a failed call launches nothing and writes nothing.
 */
#define SQUANT_NOALLOC_MAX_CTAS 32768
#define SQUANT_NOALLOC_TABLE_BYTES (256 + 8 * SQUANT_NOALLOC_MAX_CTAS)
int squant_quantize_layer_noalloc(const squant_layer *layer, const squant_options *opt,
                                  void *cuda_stream);

/*
 * Self-check of the arithmetic shortcut in SQuant-E (Algorithm 1 "Scale and SQuant-E").  The 3x3
 * path does not divide every weight by the channel's scale s; it multiplies by one correctly
 * rounded reciprocal per channel and corrects the product with two fused multiply-adds, which
 * yields the correctly rounded quotient.  This call checks that claim on the device: for each of
 * the n scales (HOST array, each in [2^-60, 2^60], the range in which the shortcut is used) it
 * runs EVERY fp32 bit pattern w with |w| <= s * qmax through both formulations and counts the
 * weights whose code or integer perturbation differ.  mismatches (HOST array of n counters) must
 * come back all zero.  Allocates and frees two small device buffers and waits for the stream.
 * About 4 ms per scale on a B200.
 */
int squant_selfcheck_division(const float *scales, int32_t n, int32_t bits, uint64_t *mismatches,
                              void *cuda_stream);

/*
 * Waits for all work on the current device and reports whether any kernel of this library gave
 * up one of its bounded waits since the last query (every wait inside the kernels - they only
 * wait for their own asynchronous copies - has an iteration limit, after which the affected
 * thread group records the fact, writes nothing and leaves).  Returns SQUANT_OK,
 * SQUANT_ERR_TIMEOUT (and clears the record) or SQUANT_ERR_CUDA.
 */
int squant_device_status(void);

/*
 * Test hooks for the failure path (no solver work).  squant_debug_set_status writes `value` into
 * the device status word that squant_device_status reads, as a kernel that gave up a wait would.
 * squant_debug_wait_expires launches one warp that waits, with a limit of max_polls (1..4096)
 * polls, on a barrier nobody arrives at: the wait runs out, the kernel records it and ends - the
 * next squant_device_status returns SQUANT_ERR_TIMEOUT and the context stays usable.
 */
int squant_debug_set_status(int value);
/*
 * The checked build of the library (libsquant_debug.so, compiled with -DSQUANT_DEBUG_BOUNDS; the
 * stand-in for a memory checker on small test cases): its kernels verify every index they form
 * into shared memory and into the launch table, and take each 3x3 channel's error sum a second
 * time from its final codes by plain division.  This call waits for the device, returns the number
 * of failed checks since the last call and the site number of the first (both 0 when all is well)
 * and clears them.  Return value: 1 if the library was built with the checks, 0 if not (the
 * counters then stay 0), or a negative error.
 */
int squant_debug_violations(int32_t *count, int32_t *first_site);
int squant_debug_wait_expires(int32_t max_polls, void *cuda_stream);

/* Number of kernels this library has launched in this process (all entry points). */
int64_t squant_launch_count(void);

/* Human readable text for an error code; never NULL. */
const char *squant_strerror(int code);

/* Text of the CUDA error behind the calling thread's last SQUANT_ERR_CUDA ("" if none). */
const char *squant_last_cuda_error(void);

/* Frees cached plans and staging buffers on all devices.  Call with no work in flight. */
int squant_shutdown(void);

#ifdef __cplusplus
}
#endif
#endif /* SQUANT_H_ */
