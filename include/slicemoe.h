/*
 * slicemoe.h - C ABI of the B200 (sm_100a) SliceMoE hot path: the MoE expert FFN computed
 * directly from bit-sliced AMAT weights (arxiv 2512.12990).
 *
 * Conventions for every entry point
 *   - Return value: 0 (SLICEMOE_OK) or a negative SLICEMOE_E_* code; slicemoe_strerror() names it.
 *     Nothing throws, aborts or prints.  Invalid arguments are rejected on the host before any
 *     launch; conditions only visible on the device (an out-of-range expert id in a device list, a
 *     wait that ran out) set bits in the status word of the workspace, see slicemoe_get_status().
 *   - "device" pointers are CUDA device memory of the current device, owned by the caller, and must
 *     stay valid until the work enqueued on `stream` has finished.  "host" pointers are ordinary
 *     host memory.  `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Unless
 *     stated, calls only enqueue work and do not synchronise.
 *   - The library allocates no device memory.
 *   - Weight matrices are row-major [N, K] (N outputs, K inputs = contraction axis); quantisation
 *     groups run along K.
 *
 * Weight format (Section 4.2 of the paper; Table 1 footnote 1: grouped asymmetric integer codes).
 *   Every weight has a b_high-bit code q; every (row, K-group) has an fp16 scale s and a u8 zero-point
 *   zp.  The code is stored as two slice planes: MSB = q >> shift (b_low bits) and LSB = q & (2^shift - 1),
 *   shift = b_high - b_low (Section 4.1: MSB and LSB slices are cached separately).  With both slices the
 *   weight is s*(q - zp); from the MSB slice alone it is 2^shift*s*((q >> shift) - (zp >> shift)), i.e. the
 *   paper's joint truncation of code and zero-point.  (b_high, b_low) is one of Table 1's three: (8, 4) -
 *   MAT84, the default everywhere - (6, 3) and (4, 2).  A plane always gives a slice value a nibble: a 3-bit
 *   or 2-bit slice sits in the low bits of its nibble, so one layout, and one set of kernels, serves the three
 *   formats; on the device MAT63 and MAT42 therefore take the bytes of MAT84.  For the slower memory tier a
 *   plane can be stored dense, 3 or 2 bits per value (slicemoe_compact_plane / slicemoe_expand_plane; the tier
 *   of slicemoe_tier_* does so).
 *
 *   Physical layout of a plane (N % 16 == 0, K % 128 == 0), N*K/2 bytes: rows are grouped in blocks
 *   of 16 and K in tiles of 64; block (rb, st) is 512 contiguous bytes at ((rb*(K/64) + st)*512),
 *   made of 32 lanes x 4 little-endian 32-bit words.  Byte j (bits 8j..8j+7) of word w of lane
 *   L = 4*g + c holds, for k = 64*st + 16*w + 4*c + j, the element (row 16*rb + g, k) in its low
 *   nibble and the element (row 16*rb + g + 8, k) in its high nibble.  Scales and zero-points are
 *   stored as [N/16][K/group][16] (row within the block fastest).  slicemoe_unpack_plane /
 *   slicemoe_unpack_meta return the canonical row-major arrays.
 */
#ifndef SLICEMOE_H
#define SLICEMOE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SLICEMOE_OK 0
#define SLICEMOE_E_INVALID_ARG (-1) /* null pointer, bad size, K % group != 0, k > E, workspace too small ... */
#define SLICEMOE_E_UNSUPPORTED (-2) /* a format or size this build does not implement */
#define SLICEMOE_E_CUDA (-3)        /* a CUDA runtime call failed */
#define SLICEMOE_E_NOMEM (-4)       /* host allocation failed (host-side objects only) */

/* Bits of the device status word (slicemoe_get_status). */
#define SLICEMOE_STATUS_BAD_EXPERT_ID 1 /* an id in a device list was outside [0, n_experts): skipped */
#define SLICEMOE_STATUS_WAIT_TIMEOUT 2  /* a bounded device-side wait ran out; the output is invalid */
#define SLICEMOE_STATUS_MISSING_LSB 4   /* both slices asked of an expert whose lsb planes are NULL: no fault; the
                                           decode output is invalid, the prefill path runs the expert MSB-only */

#define SLICEMOE_MAX_TOP_K 16
#define SLICEMOE_MAX_SHARED 4

/* One MoE layer's shape. */
typedef struct slicemoe_shape {
  int32_t hidden;              /* model width; multiple of 128, <= 4096 */
  int32_t inter;               /* routed experts' SwiGLU intermediate width; multiple of 128 */
  int32_t n_experts;           /* routed experts E */
  int32_t top_k;               /* experts per token k <= SLICEMOE_MAX_TOP_K */
  int32_t group;               /* quantisation group along K: 32, 64 or 128 */
  int32_t b_high, b_low;       /* slice configuration: (8, 4), (6, 3) or (4, 2) */
  int32_t n_shared;            /* always-on shared experts (<= SLICEMOE_MAX_SHARED), run from both slices */
  int32_t shared_inter;        /* their intermediate width; multiple of 128 */
  int32_t shared_sigmoid_gate; /* 1: shared output is scaled by sigmoid(v . x) */
} slicemoe_shape;

/* One packed weight matrix; all pointers are device pointers in the physical layout above. */
typedef struct slicemoe_mat {
  const void *msb;       /* N*K/2 bytes */
  const void *lsb;       /* N*K/2 bytes; may be NULL for a matrix that is never run at 8 bits (prec 1 for
                            such an expert is a caller error: no fault, SLICEMOE_STATUS_MISSING_LSB is set) */
  const uint16_t *scale; /* fp16 bit patterns, N*K/group entries */
  const uint8_t *zp;     /* N*K/group entries */
  int32_t N, K;
} slicemoe_mat;

/* One SwiGLU expert: gate, up [inter, hidden]; down [hidden, inter]. */
typedef struct slicemoe_expert {
  slicemoe_mat gate, up, down;
} slicemoe_expert;

const char *slicemoe_strerror(int code);
int slicemoe_version(void);
/* Text of the CUDA runtime error behind the most recent SLICEMOE_E_CUDA of this process ("no error" if none). */
const char *slicemoe_last_cuda_error(void);

/* ---- sizes ------------------------------------------------------------------------------- */
size_t slicemoe_plane_bytes(int N, int K);           /* bytes of one slice plane: N*K/2 */
size_t slicemoe_meta_count(int N, int K, int group); /* number of (scale, zp) entries: N*K/group */

/*
 * slicemoe_pack - offline preparation of one weight matrix: quantise (Table 1 fn. 1, Section 6.1:
 * grouped asymmetric codes) and split into MSB / LSB slice planes (Sections 4.1, 4.2).
 *   W      device, float32 [N, K] row-major (read only)
 *   msb, lsb, scale, zp   device outputs in the physical layout; sizes from the functions above
 * Per (row, group), in float32, with Q = 2^b_high - 1: lo = min(min w, 0), hi = max(max w, 0),
 * s = fp16((hi - lo)/Q) (round to nearest even; a group with hi == lo or s in {0, inf} gets s = 1, zp = 0),
 * zp = clamp(rint(-lo/s), 0, Q), q = clamp(rint(w/s) + zp, 0, Q) with IEEE division and
 * round-half-even.  Bit-exact and deterministic.
 * Errors: INVALID_ARG (null, N % 16, K % 128, K % group), UNSUPPORTED ((b_high, b_low) not one of (8,4), (6,3),
 * (4,2); group not in {32,64,128}), CUDA.
 */
int slicemoe_pack(const float *W, int N, int K, int group, int b_high, int b_low, void *msb,
                  void *lsb, uint16_t *scale, uint8_t *zp, void *stream);

/* Inverse of the physical layout (test hook and dump helper): nibbles[n*K + k] in 0..15. */
int slicemoe_unpack_plane(const void *plane, int N, int K, uint8_t *nibbles, void *stream);
/*
 * Dense storage of a slice plane for the slower memory tiers (Table 1: MAT63 has 3-bit slices, MAT42 2-bit ones).
 * On the device a plane gives every slice value a nibble, whatever its width; slicemoe_compact_plane writes the
 * plane's nibbles - in the order of its bytes, low nibble first - as a little-endian bit stream of `bits` bits
 * each (value i in bits [i * bits, (i + 1) * bits)), slicemoe_compact_bytes(N, K, bits) = N*K*bits/8 bytes, and
 * slicemoe_expand_plane is the inverse.  bits in {2, 3, 4} (4 is a plain copy); values must fit `bits` bits
 * (higher bits of a nibble are dropped).  plane, compact: device.  Errors: INVALID_ARG, UNSUPPORTED (bits), CUDA.
 */
size_t slicemoe_compact_bytes(int N, int K, int bits);
int slicemoe_compact_plane(const void *plane, int N, int K, int bits, void *compact, void *stream);
int slicemoe_expand_plane(const void *compact, int N, int K, int bits, void *plane, void *stream);

/* scale_rm / zp_rm: row-major [N, K/group]. */
int slicemoe_unpack_meta(const uint16_t *scale, const uint8_t *zp, int N, int K, int group,
                         uint16_t *scale_rm, uint8_t *zp_rm, void *stream);

/*
 * slicemoe_route_topk - top-k gating (Section 1) with an optional cache-priority bias (Section 2.1:
 * cache-aware routing boosts the gating scores of cached experts) and the precision request of
 * Section 4.1 (critical experts ask for both slices).
 *   logits   device float32 [T, E]
 *   bias     device float32 [E] or NULL; added to the logit in float32 for SELECTION only
 *   renorm   1: divide the k weights by their sum
 *   tau, rank_high   precision request: flag 1 (MSB+LSB) iff the expert's softmax probability
 *            (unbiased, before renormalisation) >= tau or its position in the selection < rank_high;
 *            pass tau > 1 and rank_high = 0 for "never"
 *   ids      device int32 [T, k]: experts by descending key; ties -> lower index; NaN logit = -inf
 *   weights  device float32 [T, k]: softmax(logits)[id]
 *   prec_req device uint8 [T, k] or NULL: 1 iff the float32 probability - the returned weights[t, j] when
 *            renorm = 0 - is >= tau (a float32), or j < rank_high.  The comparison is taken in float32, so the
 *            flag is an exact function of the returned weight
 * Errors: INVALID_ARG (null, T <= 0, k < 1, k > E, k > SLICEMOE_MAX_TOP_K), UNSUPPORTED (E > 512).
 */
int slicemoe_route_topk(const float *logits, int T, int E, int k, const float *bias, int renorm,
                        float tau, int rank_high, int32_t *ids, float *weights, uint8_t *prec_req,
                        void *stream);

/*
 * Workspace.  The FFN kernels need caller-owned device scratch: a header (launch count, status word, wait
 * limit), two buffers for the fp32 intermediate h (alternate launches use alternate buffers) and staging for the
 * host-buffer entry point.  Allocate slicemoe_workspace_bytes() bytes (256-byte aligned) and call
 * slicemoe_workspace_init() once before first use (it zeroes the header and marks both h buffers empty; every
 * launch leaves the workspace ready for the next).  One workspace serves one stream at a time.
 *
 * The decode kernel's CTAs (one per SM) wait for the h values that the other CTAs write, so they must all be
 * resident together.  The library refuses (UNSUPPORTED) a device on which a CTA of the kernel does not fit an SM;
 * it cannot know what else occupies the device at launch time.  If other work holds SMs for longer than the
 * wait limit (default: 10^8 clock cycles, about 50 ms), the wait for h ends by itself: the kernel returns,
 * SLICEMOE_STATUS_WAIT_TIMEOUT is set and y is not valid.  Run the decode calls on a device (or a
 * partition of it) that they have to themselves while they run, or pass SLICEMOE_COOPERATIVE to
 * slicemoe_layer_flags.  After a time-out, initialise the workspace again.
 */
size_t slicemoe_workspace_bytes(const slicemoe_shape *shape);
int slicemoe_workspace_init(void *workspace, size_t workspace_bytes, void *stream);
/* Copies the status word to *status_out (host) and clears it.  Synchronises `stream`. */
int slicemoe_get_status(void *workspace, int *status_out, void *stream);
/*
 * Sets the limit of the kernels' device-side waits for this workspace, in GPU clock cycles (0 = the default),
 * and a switch that makes the kernels treat h as never complete.  extra_arrivals is 0 in any real use; a
 * non-zero value makes the wait for h run out by construction, which is how the time-out path
 * is exercised without faulting or hanging anything: the kernel returns by itself after `wait_cycles`,
 * SLICEMOE_STATUS_WAIT_TIMEOUT is set and y is not valid.  slicemoe_workspace_init resets both.  Enqueued
 * on `stream`.
 */
int slicemoe_workspace_set_wait(void *workspace, unsigned long long wait_cycles, unsigned extra_arrivals,
                                void *stream);

/*
 * slicemoe_expert_ffn - the mixed-precision expert FFN of Section 4.1 over an expert-id/precision
 * list:   y[t] = sum_j weights[t,j] * Wd_e ( silu(Wg_e x[t]) * (Wu_e x[t]) ),  e = ids[t,j],
 * each W dequantised from both slices when prec[t,j] = 1 and from the MSB slice alone when 0.
 *   experts  device array [shape->n_experts] of slicemoe_expert
 *   x        device bf16 [T, hidden]
 *   ids, prec, weights   device [T, k] (int32, uint8, float32), k = shape->top_k
 *   y        device float32 [T, hidden], overwritten
 * Tokens are processed one after another by the batch-1 decode kernel (weights are streamed once
 * per token); accumulation is fp32, h stays fp32 between the two projections, the summation
 * order is fixed (results are bit-reproducible run to run).
 * Errors: INVALID_ARG, UNSUPPORTED (shape limits above; sum of intermediate widths over the k + n_shared
 * slots must be <= 12288; hidden / 16 must not exceed 4 x the device's SM count), CUDA.
 */
int slicemoe_expert_ffn(const slicemoe_shape *shape, const slicemoe_expert *experts, const void *x,
                        int T, const int32_t *ids, const uint8_t *prec, const float *weights,
                        float *y, void *workspace, size_t workspace_bytes, void *stream);

/*
 * slicemoe_layer - routed experts as above plus the always-on shared experts of the two evaluated
 * model architectures (not part of the paper's method): each shared expert runs from both slices and is
 * added with weight 1, or with weight sigmoid(shared_gate_vec . x[t]) when shape->shared_sigmoid_gate.
 *   shared           device array [shape->n_shared] of slicemoe_expert (inter = shape->shared_inter)
 *   shared_gate_vec  device float32 [hidden] or NULL (required iff shared_sigmoid_gate)
 */
int slicemoe_layer(const slicemoe_shape *shape, const slicemoe_expert *experts,
                   const slicemoe_expert *shared, const float *shared_gate_vec, const void *x, int T,
                   const int32_t *ids, const uint8_t *prec, const float *weights, float *y,
                   void *workspace, size_t workspace_bytes, void *stream);

/*
 * slicemoe_layer_flags - slicemoe_layer with promises from the caller that let the kernel start earlier.
 *   SLICEMOE_LISTS_RESIDENT  ids, prec and weights were complete in device memory before the work that precedes
 *            this call on `stream` began (lists uploaded by the host after its cache decision, or prepared for
 *            a whole run of layers ahead of time; NOT lists written by the kernel enqueued just before this call).
 *            The kernel then reads them, and requests the routed experts' slices, while that preceding work is
 *            still running; only x is waited for.  Results are the same bits as slicemoe_layer's.
 * Without the flag the kernel still requests the shared experts' slices early: they follow from the shape alone.
 *   SLICEMOE_COOPERATIVE  the kernel is launched as a cooperative grid: the driver guarantees that all its CTAs are
 *            resident together, or fails the launch (SLICEMOE_E_CUDA), so a device shared with other kernels
 *            cannot make the wait for h run out.  About 1.4 us per launch slower on a B200 (a cooperative grid
 *            starts as a whole, without the CTA-by-CTA hand-over from the launch before).  Same bits.
 * flags = 0 is slicemoe_layer.  Errors: as slicemoe_layer; INVALID_ARG for an unknown flag.
 */
#define SLICEMOE_LISTS_RESIDENT 1u
#define SLICEMOE_COOPERATIVE 2u
int slicemoe_layer_flags(const slicemoe_shape *shape, const slicemoe_expert *experts,
                         const slicemoe_expert *shared, const float *shared_gate_vec, const void *x, int T,
                         const int32_t *ids, const uint8_t *prec, const float *weights, float *y,
                         void *workspace, size_t workspace_bytes, unsigned flags, void *stream);

/*
 * slicemoe_layer_routed - slicemoe_route_topk and slicemoe_layer in one kernel launch per token: the decode
 * kernel's prologue computes the routing list from the router logits with the arithmetic of
 * slicemoe_route_topk (same bits), takes the precision request as the precision list (Section 4.1: experts
 * whose gating score reaches tau, or the rank_high best, run at both slices), and runs the layer.
 *   logits   device float32 [T, E]; bias, renorm, tau, rank_high as in slicemoe_route_topk
 *   ids_out, prec_out, weights_out   device [T, k] or NULL: the list the kernel used, for the caller's cache
 *            bookkeeping (written by one CTA; valid when the call's work on `stream` has completed)
 * A caller whose slice cache may override the request (a missing LSB slice) uses the two separate calls.
 * Errors: as slicemoe_layer, plus UNSUPPORTED for E > 512.
 */
int slicemoe_layer_routed(const slicemoe_shape *shape, const slicemoe_expert *experts,
                          const slicemoe_expert *shared, const float *shared_gate_vec, const void *x, int T,
                          const float *logits, const float *bias, int renorm, float tau, int rank_high,
                          int32_t *ids_out, uint8_t *prec_out, float *weights_out, float *y,
                          void *workspace, size_t workspace_bytes, void *stream);

/*
 * slicemoe_trace_read - time stamps of the decode kernel's most recent launch, for a library built with
 * -DSLICEMOE_TRACE (python -m paper_2512_12990_b200.build --trace builds libslicemoe_trace.so beside the ordinary
 * library; python -m paper_2512_12990_b200.trace prints the timeline).  out_host: host array
 * [min(max_ctas, 256)][*slots_out] of int64: clock64 since the CTA's start at the points the source lists, and the
 * global timer at three of them; *slots_out is at most 256, so 256 * 256 entries always suffice.  Synchronises the
 * device.  The ordinary build returns UNSUPPORTED.
 */
int slicemoe_trace_read(long long *out_host, int max_ctas, int *slots_out);

/*
 * slicemoe_stream_probe - a measuring stick, not part of the method: brings exactly the bytes that one
 * slicemoe_layer call with T = 1 reads for this list - MSB plane, LSB plane where prec = 1, scales and zero-points
 * of gate, up and down of every listed expert, and of the shared experts at 8 bits - into shared memory with the
 * decode kernel's bulk copies (16 KB each, one CTA per SM, twelve copies in flight per CTA) and does nothing with
 * them.  Its time per launch is what the memory system alone needs for a decode step of the layer.
 *   ids, prec   device [top_k]; entries outside [0, n_experts) are skipped
 *   dependent   1: no byte is requested before the work ahead on `stream` has completed (a kernel all of whose
 *               input depends on its predecessor); 0: the lists must be resident in the sense of
 *               SLICEMOE_LISTS_RESIDENT, and launches overlap as far as the hardware lets them
 *   bytes_out_device   device, or NULL: the bytes of the step are ADDED to it (one CTA does)
 *   status_out_device  device int32, or NULL: set to 1 if a (bounded) wait for a copy ran out
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA.
 */
int slicemoe_stream_probe(const slicemoe_shape *shape, const slicemoe_expert *experts,
                          const slicemoe_expert *shared, const int32_t *ids, const uint8_t *prec,
                          int dependent, unsigned long long *bytes_out_device, int *status_out_device,
                          void *stream);

/*
 * slicemoe_layer_static - slicemoe_layer for callers that cannot allocate device memory.  (The paper
 * has no counterpart; this is a convenience of the library.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a host callback or another
 * context where the CUDA runtime forbids allocation, under a memory pool that owns every byte of the
 * device, or in a plug-in that receives input and output buffers from its host application and has
 * no allocator of its own.  Such a caller cannot provide the workspace that slicemoe_layer asks for,
 * so this variant keeps the workspace inside the library: a fixed array of 127,168 bytes in device
 * memory that every GPU holds from the moment it loads the library until the process exits.
 *
 * Arguments are those of slicemoe_layer without workspace / workspace_bytes; inputs and outputs are
 * still the caller's.  The computation and its result are the same as slicemoe_layer's.
 *   - Limits: the array is sized for hidden <= 4096 and top_k * inter + n_shared * shared_inter <= 12288
 *     (the limits of slicemoe_layer itself).  A larger layer is refused with SLICEMOE_E_UNSUPPORTED;
 *     nothing is ever allocated to make it fit.
 *   - The call allocates nothing and frees nothing, directly or through any library.
 *   - First call on a device: the library looks up the device address of its array once per device
 *     (with that device current) and remembers it.  Make this first call outside any stream capture, and
 *     from one host thread (the look-up is not guarded against a second thread doing the same at once).
 *   - The array is shared by all calls on a device and keeps the previous call's contents; each call
 *     clears the part that must start at zero (on `stream`, before its kernels).  Two calls whose work
 *     overlaps on the GPU - different streams, or different host threads without ordering - race on
 *     it and give undefined results: keep calls on one device ordered one after the other.
 *   - The device status word lives in the same array and is not readable through this entry point;
 *     use slicemoe_layer with your own workspace if you need slicemoe_get_status.
 * Errors: as slicemoe_layer.
 */
int slicemoe_layer_static(const slicemoe_shape *shape, const slicemoe_expert *experts,
                          const slicemoe_expert *shared, const float *shared_gate_vec, const void *x,
                          int T, const int32_t *ids, const uint8_t *prec, const float *weights,
                          float *y, void *stream);

/*
 * slicemoe_decode_step_host - one batch-1 decode step of a layer with HOST inputs and outputs:
 * copies x (bf16 [hidden]) and logits (float32 [E]) to the device, runs slicemoe_layer_routed
 * (bias/tau/rank_high as in slicemoe_route_topk; the precision request is used as the precision
 * list), copies y (float32 [hidden]) back and synchronises `stream`.  x_host, logits_host
 * and y_host should be pinned for the copies to be asynchronous.  logits_host may be NULL: the logits then
 * follow x directly in the buffer at x_host (bf16 [hidden], then float32 [E]) and one copy brings both.  When y_host is pinned,
 * device-mapped host memory (cudaHostAlloc / cudaHostRegister, 16-byte aligned) the kernel writes y
 * straight into it and no copy back is issued.  Weights stay resident on the device.  Staging
 * buffers live in the workspace.
 */
int slicemoe_decode_step_host(const slicemoe_shape *shape, const slicemoe_expert *experts,
                              const slicemoe_expert *shared, const float *shared_gate_vec,
                              const void *x_host, const float *logits_host, const float *bias,
                              int renorm, float tau, int rank_high, float *y_host, void *workspace,
                              size_t workspace_bytes, void *stream);

/*
 * slicemoe_prefill_layer - the layer for a prompt of T tokens at once (Section 3: prefill visits
 * every expert of a layer, so the expert FFN becomes a grouped dense contraction).  Section 6.3 says that
 * prefill wants high-bit computation; the per-expert precision flag is this library's generalisation (an
 * expert may also be run from its MSB slice alone), which a mixed-precision prefill uses.
 * Tokens are grouped by expert on the device; per 128-token tile the weight tile is dequantised
 * from the nibble planes - s*(q - zp), or 16*s*(q_msb - (zp >> 4)) for an MSB-only expert - into
 * tensor memory as the exact sum of two fp16 numbers per weight (no weight is rounded) and
 * contracted on the tensor cores (tcgen05, fp16 x fp16 with fp32 accumulation); tokens enter as
 * fp16 (exact for bf16 inputs in fp16's normal range) and h is rounded to fp16 between the two
 * projections (relative error 2^-11, inside the FFN tolerance).  Both conversions go to fp16's range: a token
 * value or an h beyond +-65504 becomes infinite and that row of y is not finite (nothing faults, no status
 * bit is set); activations of that size do not occur behind a normalisation layer.  Each
 * (token, expert) pair gets its own fp32 result row and y[t] sums them in list order (routed
 * slots 0..k-1, then the shared experts), so y is bit-reproducible run to run.
 *   x            device bf16 [T, hidden]
 *   shared_gate_vec  as for slicemoe_layer; 8-byte aligned
 *   ids, weights device [T, k] (int32, float32)
 *   expert_prec  device uint8 [n_experts]: 1 = both slices, 0 = MSB slice only.  Precision is per
 *                expert, not per (token, slot): all tokens of an expert share its weight tile.
 *                Shared experts always use both slices.
 *   y            device float32 [T, hidden], overwritten; 16-byte aligned
 *   workspace    device, >= slicemoe_prefill_workspace_bytes(shape, T) bytes, 256-byte aligned; holds
 *                the token lists, the gathered x and h (fp16) and the per-pair result rows (fp32).
 *                Needs no initialisation; contents are scratch.
 *   status_out_device  device int32, overwritten: OR of SLICEMOE_STATUS_BAD_EXPERT_ID (a pair whose id
 *                is outside [0, E) is skipped) and SLICEMOE_STATUS_MISSING_LSB (expert_prec 1 for an
 *                expert without LSB planes: it runs MSB-only) and SLICEMOE_STATUS_WAIT_TIMEOUT (a bounded wait
 *                inside the GEMM kernel ran out: y is not valid).
 * Shape limits: hidden, inter, shared_inter multiples of 128 (no upper limit on hidden here);
 * T * (k + n_shared) <= 2^28.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA.  slicemoe_prefill_workspace_bytes returns 0 for a shape or T
 * that slicemoe_prefill_layer would refuse.
 */
size_t slicemoe_prefill_workspace_bytes(const slicemoe_shape *shape, int T);
int slicemoe_prefill_layer(const slicemoe_shape *shape, const slicemoe_expert *experts,
                           const slicemoe_expert *shared, const float *shared_gate_vec, const void *x,
                           int T, const int32_t *ids, const float *weights, const uint8_t *expert_prec,
                           float *y, void *workspace, size_t workspace_bytes, int *status_out_device,
                           void *stream);

/*
 * Host-side Dynamic Bit-Sliced Caching bookkeeping (Section 4.1; cache set-up of Section
 * 6.1).  Pure host code: it only turns (expert id, precision request) lists into the precision
 * list the FFN runs with, plus hit/miss accounting.  MSB slices: LRU.  LSB slices: lowest priority,
 * evicted (oldest first) before any MSB slice.  One cache for all layers.  Optional miss budget:
 * once step >= warmup_steps, while bytes fetched / full-precision bytes of the same requests
 * exceeds miss_budget, an LSB miss is not fetched and the expert runs MSB-only.
 */
typedef struct slicemoe_dbsc slicemoe_dbsc;
/* miss_budget < 0 disables the budget.  Returns NULL on allocation failure or bad arguments. */
slicemoe_dbsc *slicemoe_dbsc_create(int64_t capacity_bytes, int64_t msb_bytes, int64_t lsb_bytes,
                                    double miss_budget, int warmup_steps);
void slicemoe_dbsc_destroy(slicemoe_dbsc *c);
/* Serves one selected expert.  Returns the execution precision (1 = MSB+LSB, 0 = MSB only) or a
 * negative error.  msb_hit / lsb_hit (nullable): 1 hit, 0 miss, -1 (lsb only) not requested.
 * fetched_bytes (nullable): bytes this request had to fetch. */
int slicemoe_dbsc_request(slicemoe_dbsc *c, int step, int layer, int expert, int need_lsb,
                          int *msb_hit, int *lsb_hit, int64_t *fetched_bytes);
/* Serves n selected experts of one (step, layer) in list order: prec_out[i] for ids[i] with request
 * prec_req[i].  All host pointers. */
int slicemoe_dbsc_assign(slicemoe_dbsc *c, int step, int layer, const int32_t *ids,
                         const uint8_t *prec_req, int n, uint8_t *prec_out);
#define SLICEMOE_DBSC_NSTATS 12
/* out[0..11] = requests, msb_hit, msb_miss, lsb_hit, lsb_miss, lsb_skipped, bytes_fetched,
 * high_exec, low_exec, win_bytes_fetched, win_bytes_full, bytes_used. */
int slicemoe_dbsc_stats(const slicemoe_dbsc *c, int64_t *out);
/* 1/0 presence of the two slices of (layer, expert). */
int slicemoe_dbsc_contains(const slicemoe_dbsc *c, int layer, int expert, int *has_msb, int *has_lsb);

/*
 * For a caller that keeps the slices themselves (slicemoe_tier_* below): with logging on, every slice that a
 * request evicts is remembered until slicemoe_dbsc_drain_evicted hands it out (layer, expert, 1 for an LSB slice;
 * at most `max` per call, oldest first; returns how many were written, or a negative error).
 */
int slicemoe_dbsc_log_evictions(slicemoe_dbsc *c, int on);
int slicemoe_dbsc_drain_evicted(slicemoe_dbsc *c, int32_t *layers, int32_t *experts, uint8_t *is_lsb, int max);

/*
 * A second memory tier under the slice cache (Section 5: the full set of weights lives in a large, slow store
 * and is touched only when a slice misses).  The slow store is pinned host memory, the fast tier a pool of
 * equal slots in device memory, a miss a copy of the slice's record on a side stream; the decisions are those
 * of slicemoe_dbsc_* (MSB slices LRU, LSB slices first to go), with both slice kinds charged one slot.
 *
 * Records.  MSB record: gate MSB plane, gate scales, gate zero-points, then up's, then down's.  LSB record:
 * gate, up, down LSB planes.  In the store a plane of a slice narrower than four bits (MAT63: 3 + 3, MAT42:
 * 2 + 2) is kept dense, as slicemoe_compact_plane writes it, so a miss moves 3 or 2 bits per weight instead of 4;
 * the copy lands in a staging buffer and a small kernel on the side stream spreads it into the slot's nibble
 * planes.  slicemoe_tier_sizes gives, for a shape: the stored sizes of the two records, the slot size (the larger
 * record in its device form, rounded up to 256 bytes) and the staging size (0 for MAT84, whose records are
 * stored as they are used).  The store holds for (layer l, expert e) the MSB record followed by the LSB record
 * at offset (l * n_experts + e) * (msb_record + lsb_record); slicemoe_tier_store_expert writes one such pair from a
 * packed expert on the device (device-to-host copies enqueued on `stream`; scratch_device: device memory of the
 * staging size, NULL for MAT84; offline preparation).
 *
 * slicemoe_tier_create: store_host (pinned, read only, must outlive the tier); pool_device (256-byte aligned,
 * pool_bytes >= (1 + 4 * top_k) slots: slot 0 is a stand-in that the table entries of non-resident slices point
 * to, so that a list naming an expert that was never requested reads defined bytes); tables_device: device array
 * [n_layers * n_experts] of slicemoe_expert that the tier fills and keeps up to date - pass
 * tables_device + l * n_experts as `experts` to the layer calls; staging_device: device memory of at least the
 * staging size (16-byte aligned; NULL for MAT84).  Synchronises `stream`.  NULL on bad arguments
 * or allocation failure.  The tier allocates no device memory.
 *
 * slicemoe_tier_request: serves the n selected experts of one (step, layer): decides hits, misses, evictions
 * and the execution precision (prec_out, host), copies missing records into free slots on `copy_stream` - after
 * everything already enqueued on `compute_stream` has finished, so that no slice still being read is
 * overwritten - updates the device tables, and makes `compute_stream` wait for the copies.  The next layer
 * call on compute_stream with ids / prec_out then finds every slice it reads in the pool: a slice of the list
 * that a later entry of the same list pushed out of the cache's books again keeps its bytes until the next
 * request (2 * top_k slots of the pool are set aside for that; the cache is given the rest less slot 0).  ids,
 * prec_req, prec_out are host arrays.  Errors: INVALID_ARG, UNSUPPORTED (the pool cannot hold the list), NOMEM, CUDA.
 *
 * slicemoe_tier_sync: makes the pool hold exactly what the cache's books hold - for use after the books were
 * changed behind the tier's back, which is how Predictive Cache Warmup (Section 4.3) reaches the tier: call
 * slicemoe_dbsc_prefill_layer / _end on slicemoe_tier_cache(t) while the prompt is prefilled, then
 * slicemoe_tier_sync once, and the decode steps that follow find the warmed slices in the pool.  Streams as in
 * slicemoe_tier_request.  (What is not modelled is the traffic of the warm-up itself while the prompt is still
 * running: the slices arrive in one go at the end.)
 */
typedef struct slicemoe_tier slicemoe_tier;
int slicemoe_tier_sizes(const slicemoe_shape *shape, size_t *msb_record, size_t *lsb_record, size_t *slot_bytes,
                        size_t *staging_bytes);
int slicemoe_tier_store_expert(const slicemoe_shape *shape, const slicemoe_expert *expert, void *record_host,
                               void *scratch_device, void *stream);
slicemoe_tier *slicemoe_tier_create(const slicemoe_shape *shape, int n_layers, const void *store_host,
                                    void *pool_device, size_t pool_bytes, slicemoe_expert *tables_device,
                                    void *staging_device, size_t staging_bytes, double miss_budget,
                                    int warmup_steps, void *stream);
void slicemoe_tier_destroy(slicemoe_tier *t);
slicemoe_dbsc *slicemoe_tier_cache(slicemoe_tier *t); /* the tier's own cache, for statistics; owned by the tier */
int slicemoe_tier_request(slicemoe_tier *t, int step, int layer, const int32_t *ids, const uint8_t *prec_req,
                          int n, uint8_t *prec_out, void *compute_stream, void *copy_stream);
int slicemoe_tier_sync(slicemoe_tier *t, void *compute_stream, void *copy_stream);
int slicemoe_tier_stats(const slicemoe_tier *t, int64_t *bytes_copied, int64_t *copies, int64_t *free_slots);

/*
 * The cache-aware routing baselines the paper compares with (Section 2.1; Section 6.1, "Baseline MoE
 * Acceleration").  The paper names them without formulas; what is implemented:
 * slicemoe_dbsc_bias - Cache-Prior: bias_out[e] (host float32 [n_experts]) = delta if the MSB slice of
 *   (layer, e) is resident, else 0: the `bias` input of slicemoe_route_topk, which uses it for selection only.
 * slicemoe_cumsum_select - Cumsum: experts ranked by descending probability (ties: lower index); the candidate
 *   set is the shortest prefix of the ranking that holds at least k experts and a probability mass of at least p;
 *   cached candidates (cached[e] != 0) are selected first, then the others, each in ranking order, k in all.
 *   probs, cached: host [n_experts]; ids_out: host int32 [k].
 * Errors: INVALID_ARG, NOMEM.
 */
int slicemoe_dbsc_bias(const slicemoe_dbsc *c, int layer, int n_experts, float delta, float *bias_out);
int slicemoe_cumsum_select(const float *probs, const uint8_t *cached, int n_experts, int k, double p,
                           int32_t *ids_out);

/*
 * The hardware cost model of Section 5 (System Implementation), as used for the energy and speed-up figures of
 * Section 6.3.  Host arithmetic only.  The paper prints the constants, not the model; the model here:
 *   energy  = 8 flash_bytes (flash_pj + dram_pj) + 8 dram_bytes dram_pj   [pJ]  + 2 macs / tops_per_watt
 *             (a byte that comes from Flash is also written to DRAM once)
 *   latency = 8 flash_bytes / flash_gbps + max(8 dram_bytes / dram_gbps, 2 macs / tops)
 *             (a missed slice arrives before its expert runs; DRAM reads stream under the computation)
 * slicemoe_cost_paper_hw fills in the paper's numbers: 1.5 and 103 pJ/bit, 104 and 10 Gbps, 16.4 TOPS,
 * 3.18 TOPS/W.  energy_joule / latency_s may be NULL.  Errors: INVALID_ARG.
 */
typedef struct slicemoe_cost_hw {
  double dram_pj_per_bit, flash_pj_per_bit; /* energy per bit read or written */
  double dram_gbps, flash_gbps;             /* bandwidth in 10^9 bit/s */
  double tops, tops_per_watt;               /* 10^12 operations per second, and per joule */
} slicemoe_cost_hw;
void slicemoe_cost_paper_hw(slicemoe_cost_hw *hw);
int slicemoe_cost_step(const slicemoe_cost_hw *hw, int64_t flash_bytes, int64_t dram_bytes, int64_t macs,
                       double *energy_joule, double *latency_s);

/*
 * Predictive Cache Warmup (Section 4.3): the cache is reshaped while a prompt is prefilled, so that decode
 * starts with the slices it is likely to ask for.  Call slicemoe_dbsc_prefill_layer once per layer, in the
 * order prefill visits them, with the layer's routing result, then slicemoe_dbsc_prefill_end.
 *   ids, scores  host [n_pairs] (= tokens x top-k, any order): selected expert and its gating score
 *   tau          the threshold that makes an expert critical in decode
 * Per expert the call takes the number of pairs (access frequency) and the mean score (double sum in list
 * order / count).  Every expert with frequency > 0 gets its MSB slice into the cache, and its LSB slice if
 * its mean score >= tau.  While the content exceeds the capacity, LSB slices are dropped in ascending
 * (score, frequency, layer, expert) order, then MSB slices in ascending (frequency, score, layer, expert)
 * order; slices that were cached before the prompt (no statistics) go before any of the prompt's, LSB
 * then MSB.  prefill_end re-orders
 * both lists by the same keys (the most frequent MSB slice becomes the most recently used) and forgets the
 * statistics.  Hit/miss counters are not touched: prefill loads every expert it uses anyway (Section 3).
 * Errors: INVALID_ARG (null, negative layer or count, an id outside [0, n_experts)), NOMEM.
 */
int slicemoe_dbsc_prefill_layer(slicemoe_dbsc *c, int layer, const int32_t *ids, const float *scores,
                                int64_t n_pairs, int n_experts, double tau);
int slicemoe_dbsc_prefill_end(slicemoe_dbsc *c);

#ifdef __cplusplus
}
#endif
#endif /* SLICEMOE_H */
