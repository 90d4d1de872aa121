/*
 * hq.h - C ABI of the B200 (sm_100a) library for HAWQ-V3 integer-only inference.
 *
 * Every entry point works on DEVICE memory unless its comment says otherwise.  The caller owns
 * all tensors, weights, biases and dyadic arrays and keeps them alive until the work queued on
 * `stream` has finished.  The library allocates only inside hq_handle / hq_network objects and
 * frees that memory in the matching destroy call.  Calls are asynchronous on `stream` (a
 * cudaStream_t passed as void*; NULL = the legacy default stream).  Argument and launch errors
 * come back synchronously as hq_status; a device-side wait that ran out of its bounded budget is
 * reported by hq_sync().  Nothing aborts, throws or prints.  There is no CPU fallback: a shape
 * the kernels cannot run returns HQ_ERR_UNSUPPORTED.
 *
 * Conventions
 *   - activations are dense NHWC; weights are [cout][kh][kw][cin], signed;
 *   - bits == 4 tensors hold two values per byte along the channel axis: channel 2j in bits 3:0
 *     of byte j, channel 2j+1 in bits 7:4, signed values in two's complement; c must be even;
 *   - activations have zero point 0, so spatial padding is the integer 0;
 *   - `data` pointers are 16-byte aligned, otherwise HQ_ERR_ALIGNMENT;
 *   - input and output of a call must not overlap.
 *
 * Integer semantics (identical for all entry points), with Int(.) = round-half-up:
 *   dn(q, b, c) = (q * b + 2^(c-1)) >> c      64-bit product, arithmetic shift, 1 <= c <= 62,
 *                                             0 <= b < 2^31: the dyadic number b / 2^c applied
 *                                             to an INT32 value (Eq. 4 and the DN(.) definition).
 */
#ifndef HQ_H_
#define HQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hq_handle hq_handle;   /* opaque: device, status word, workspace */
typedef struct hq_network hq_network; /* opaque: a planned layer table */

typedef enum {
  HQ_OK = 0,
  HQ_ERR_INVALID_ARG = 1,  /* null pointer, bad dimension, bits/sign/clamp combination */
  HQ_ERR_UNSUPPORTED = 2,  /* valid request no kernel covers */
  HQ_ERR_ALIGNMENT = 3,    /* a data pointer is not 16-byte aligned */
  HQ_ERR_RANGE = 4,        /* reserved: accumulator + bias left INT32 (the CPU oracle reports it) */
  HQ_ERR_WORKSPACE = 5,    /* device allocation failed, or the request exceeds a fixed scratch array */
  HQ_ERR_CUDA = 6,         /* a CUDA runtime or driver call failed */
  HQ_ERR_TIMEOUT = 7,      /* a bounded device-side wait expired; outputs are not valid */
  HQ_ERR_INFEASIBLE = 8    /* hq_ilp_solve: no assignment meets the limits */
} hq_status;

typedef struct {  /* activation tensor, dense NHWC */
  void* data;     /* device pointer, caller-owned */
  int32_t n, h, w, c; /* logical extents; bits == 4 needs c even */
  int32_t bits;       /* 4, 8 or 32 */
  int32_t is_signed;  /* 0: values in [0, 2^bits-1]; 1: two's complement (always 1 for 32) */
} hq_tensor;

typedef struct {    /* per-channel dyadic pairs b / 2^c, two device arrays of the channel count */
  const int32_t* b; /* 0 <= b < 2^31 */
  const int32_t* c; /* 1 <= c <= 62 */
} hq_dyadic;

typedef struct {
  int32_t kh, kw, stride, pad, cin, cout;
  int32_t w_bits;      /* 8 or 4; must equal the input tensor's bits (Section 3.4: b_w == b_a) */
  const void* w;       /* [cout][kh][kw][cin] signed, 4-bit packed along cin */
  const int32_t* bias; /* [cout] INT32 at scale S_h * S_w[oc] (Appendix D); NULL means 0 */
  hq_dyadic requant;   /* DN(S_w[oc] S_h / S_a); ignored when the output has bits == 32 */
  const hq_tensor* residual; /* NULL, or a tensor with the output's n,h,w,c and bits 8 or 32 */
  hq_dyadic res_rescale;     /* DN(S_r / S_a) as arrays of length cout; used with residual */
  int32_t relu;              /* applied after the residual add */
  int32_t qmin, qmax;        /* clamp bounds, inside the output type's range */
} hq_conv_desc;

#define HQ_CONCAT_MAX_BRANCHES 8

typedef enum {
  HQ_OP_CONV = 0,    /* hq_conv2d; in1 = residual tensor id or -1 */
  HQ_OP_LINEAR = 1,  /* hq_linear on the flattened input */
  HQ_OP_MAXPOOL = 2, /* hq_maxpool */
  HQ_OP_AVGPOOL = 3, /* hq_avgpool_requant with `rescale0` */
  HQ_OP_ADD = 4,     /* hq_residual_add(in0 by rescale0, in1 by rescale1) */
  HQ_OP_REQUANT = 5, /* hq_residual_add with no second operand */
  HQ_OP_CONCAT = 6,  /* hq_concat_requant over the tensors ins[0 .. n_in) with the pairs rescales[] (Appendix E) */
  HQ_OP_SUMPOOL = 7  /* hq_sumpool of in0 with pool_k / pool_stride / pool_pad: INT32 window sums (Appendix E) */
} hq_op;

typedef struct {       /* one row of the per-layer table; layer i produces tensor id i */
  int32_t op;          /* hq_op */
  int32_t in0, in1;    /* tensor ids: -1 = the network input image (in0) / none (in1) */
  hq_conv_desc conv;   /* CONV / LINEAR: geometry, bit-width, device pointers; .residual ignored */
  hq_dyadic rescale0;  /* AVGPOOL / ADD / REQUANT: pair applied to in0 */
  hq_dyadic rescale1;  /* ADD: pair applied to in1 */
  int32_t pool_k, pool_stride, pool_pad; /* MAXPOOL */
  int32_t out_bits, out_signed;          /* type of the produced tensor */
  int32_t relu, qmin, qmax;              /* AVGPOOL / ADD / REQUANT / CONCAT (CONV uses conv.*) */
  int32_t n_in;                          /* CONCAT: number of branches, 1 .. HQ_CONCAT_MAX_BRANCHES */
  int32_t ins[8];                        /* CONCAT: tensor ids of the branches, in channel order */
  hq_dyadic rescales[8];                 /* CONCAT: DN(S_i / S_a) of branch i, arrays of that branch's channel count */
} hq_layer;

/* Create / destroy the per-device context.  `device` is a CUDA ordinal.  Host call.
 * A handle owns small device buffers that its calls reuse (a status word, scratch for lowered or widened
 * operands, the narrow multiply-add pairs of a large element-wise call): calls through ONE handle must be
 * ordered on the device (one stream, or streams joined by events); use one handle per concurrent stream. */
hq_status hq_create(int32_t device, hq_handle** out);
hq_status hq_destroy(hq_handle* h);

/* Wait for `stream` and report HQ_ERR_TIMEOUT if any kernel launched through `h` gave up a
 * bounded wait since the last hq_sync (the status word is cleared). */
hq_status hq_sync(hq_handle* h, void* stream);

/*
 * Quantized convolution with the fused integer epilogue (Section 3.1, Eq. 3-4; Section 3.2 /
 * Appendix D for the bias; Section 3.3 and Appendix G for the residual):
 *   acc = sum_{r,s,ci} in[n, oh*stride+r-pad, ow*stride+s-pad, ci] * w[oc,r,s,ci]   (INT32)
 *   t   = acc + bias[oc]
 *   out->bits == 32 :  out = t
 *   otherwise       :  y = dn(t, b[oc], c[oc]);  if residual: y += dn(res, rb[oc], rc[oc]);
 *                      if relu: y = max(y, 0);  out = clamp(y, qmin, qmax), stored at out->bits.
 * in: bits 8 or 4 (== w_bits), signed or unsigned.  out: n, h, w, c must equal the convolution's
 * output extents.  The tensor-core kernel takes layers with cin a multiple of 32, directly or - for the
 * 3-channel first layer, thin layers and layers whose input tensor is below 128 KiB - through a lowered form
 * (space-to-depth copy or patch matrix in scratch memory of the handle); other shapes run on the CUDA-core
 * path.  Accumulator overflow beyond INT32
 * is undefined (cannot happen for K = kh*kw*cin <= 66311 with 8-bit operands).
 */
hq_status hq_conv2d(hq_handle* h, const hq_tensor* in, const hq_conv_desc* desc, hq_tensor* out, void* stream);

/* Fully connected layer = hq_conv2d with kh = kw = 1 on an (n,1,1,c) tensor (Eq. 3 as a matrix
 * product).  `desc` must have kh = kw = stride = 1, pad = 0, residual = NULL. */
hq_status hq_linear(hq_handle* h, const hq_tensor* in, const hq_conv_desc* desc, hq_tensor* out, void* stream);

/*
 * Integer residual add on stored tensors (Section 3.3): per element of channel ch
 *   y = dn(main, mb[ch], mc[ch]) + (res ? dn(res, rb[ch], rc[ch]) : 0); ReLU; clamp; store.
 * Each branch is rounded on its own and then added (Appendix G).  main/res: bits 4, 8 or 32;
 * out: bits 4, 8 or 32 (32: the sum stays INT32, the wide residual stream of Fig. 2, clamped to [qmin, qmax]).
 * res == NULL gives a plain dyadic requantization.
 */
hq_status hq_residual_add(hq_handle* h, const hq_tensor* main_t, hq_dyadic main_rescale,
                          const hq_tensor* res, hq_dyadic res_rescale,
                          int32_t relu, int32_t qmin, int32_t qmax, hq_tensor* out, void* stream);

/*
 * Global average pooling on wide integers with no division (Appendix E; Section 1 on avoiding
 * integer division): sum over the h*w pixels in INT32, then clamp(dn(sum, b[ch], c[ch])), the
 * factor 1/(h*w) being part of b / 2^c.  in: (n,h,w,c) bits 4/8/32; out: (n,1,1,c) bits 4/8.
 */
hq_status hq_avgpool_requant(hq_handle* h, const hq_tensor* in, hq_dyadic rescale,
                             int32_t qmin, int32_t qmax, hq_tensor* out, void* stream);

/*
 * Concatenation along the channel axis with a dyadic rescale per branch (Appendix E, concatenation
 * layer: every branch of an Inception module gets its own DN rescale to the output scale before the
 * channel ranges are joined):
 *   out[n,h,w, off_i + k] = clamp(relu?(dn(branch_i[n,h,w,k], b_i[k], c_i[k]))),  off_i = c_0 + ... + c_{i-1}.
 * `branches` and `rescale` are HOST arrays of n_branches entries (1 <= n_branches <=
 * HQ_CONCAT_MAX_BRANCHES); each tensor's data and each pair's b / c arrays (length = that branch's
 * channel count) are DEVICE pointers, caller-owned.  Branch bits: 4, 8 or 32 (the paper keeps the
 * pooling branch in INT32); all branches share out's n, h, w and their channel counts sum to out->c.
 * out: bits 8, or 4 when every branch has an even channel count (else HQ_ERR_UNSUPPORTED).  One launch,
 * asynchronous on `stream`; every operand is read once and the output written once.
 */
hq_status hq_concat_requant(hq_handle* h, int32_t n_branches, const hq_tensor* branches, const hq_dyadic* rescale,
                            int32_t relu, int32_t qmin, int32_t qmax, hq_tensor* out, void* stream);

/*
 * k x k window SUMS on wide integers (Appendix E keeps the pooling layer, i.e. the pooling branch of
 * an Inception module, on the INT32 feature map):
 *   out[n,oh,ow,c] = sum_{r,s < k} in[n, oh*stride+r-pad, ow*stride+s-pad, c], taps outside the image = 0.
 * An average pool is this sum followed by a dyadic pair that carries 1/k^2 (hq_concat_requant,
 * hq_residual_add): no division (Section 1).  in: bits 4, 8 or 32; out: bits 32, extents
 * (h + 2 pad - k) / stride + 1.  pad < k.  Sums beyond INT32 are undefined (the oracle reports them).
 */
hq_status hq_sumpool(hq_handle* h, const hq_tensor* in, int32_t k, int32_t stride, int32_t pad,
                     hq_tensor* out, void* stream);

/* k x k max pooling of an 8-bit or INT32 tensor (Appendix E pools on the wide feature map); window taps outside
 * the image are ignored (ResNet stem; an integer max commutes with the monotone requantization of Eq. 4).  pad < k. */
hq_status hq_maxpool(hq_handle* h, const hq_tensor* in, int32_t k, int32_t stride, int32_t pad,
                     hq_tensor* out, void* stream);

/*
 * Plan a network from its per-layer table (bit-widths, geometry, dyadic pairs, residual wiring;
 * Fig. 2 dataflow in fused form, first and last layer 8-bit per Appendix H).  `table` is a HOST
 * array; the pointers inside it are DEVICE pointers that must outlive the network.  Activation
 * buffers for `batch` images of image_h x image_w x image_c (8-bit) are allocated here.
 */
hq_status hq_network_create(hq_handle* h, const hq_layer* table, int32_t n_layers, int32_t batch,
                            int32_t image_h, int32_t image_w, int32_t image_c, int32_t image_signed,
                            hq_network** out);

/*
 * Run the table on `images` (device, NHWC 8-bit, the planned batch) and write the last layer's
 * output to `logits` (device; its n,c,bits must match the last layer).  `layer_taps` is NULL or
 * a HOST array of n_layers device pointers (NULL entries allowed) that receive a copy of each
 * layer's output in its stored format.
 */
hq_status hq_run_network(hq_network* net, const hq_tensor* images, hq_tensor* logits,
                         void* const* layer_taps, void* stream);

/* Measurement aid: run the table once with plain launches and a CUDA event pair around every
 * layer, wait for the stream, and write each layer's device time in nanoseconds to the HOST
 * array ns[n_layers]. */
hq_status hq_network_time_layers(hq_network* net, const hq_tensor* images, hq_tensor* logits, int64_t* ns,
                                 void* stream);

/* Measurement aid: the contraction of Eq. 3 alone.  Launches one kernel (asynchronous on `stream`) in which every
 * SM issues `rounds` x `blocks_per_round` blocks of four tcgen05.mma kind::i8 instructions (128 x 256 x 32, s8 x u8 ->
 * s32) back to back from pseudo-random operands resident in shared memory, with no loads and no epilogue, and
 * writes the integer operations of the launch (2 per multiply-accumulate) to *ops (HOST, may be NULL).  Timed by the
 * caller (events on `stream`); hq_sync reports an expired wait.  rounds in [1, 2^20], blocks_per_round in [1, 2^16]. */
hq_status hq_mma_peak_launch(hq_handle* h, int32_t rounds, int32_t blocks_per_round, int64_t* ops, void* stream);

/* Bytes of layer i's stored output and the number of kernels one hq_run_network launches. */
hq_status hq_network_layer_bytes(const hq_network* net, int32_t layer, int64_t* bytes);
hq_status hq_network_launch_count(const hq_network* net, int32_t* launches);
hq_status hq_network_destroy(hq_network* net);

/* Debug aid (no paper counterpart): every device buffer a network owns - layer outputs, widened weights,
 * scratch - lies between two 256-byte guard bands written when the network is built.  This call waits for
 * `stream`, reads the bands back and returns HQ_ERR_RANGE if any byte changed, with the layer that owns the
 * buffer in *bad_layer (-1: the shared scratch buffer; bad_layer may be NULL): a kernel wrote before the
 * first or beyond the last byte of a tensor.  Host call; HQ_OK means every band is intact. */
hq_status hq_network_check_guards(const hq_network* net, void* stream, int32_t* bad_layer);

/*
 * hq_conv2d for callers that cannot allocate device memory.  (The paper has no counterpart: this is
 * a deployment convenience of the library, not a step of the method.)
 *
 * Who this is for: code that must not call cudaMalloc when a layer runs - a serving process whose
 * memory was carved up at start-up and whose policy forbids later driver allocations (they stall
 * every stream of the context and can fail under a tight budget), a component running while another
 * library owns the rest of the device memory, or a plug-in that was handed a stream and buffers
 * but no allocator.  hq_conv2d may grow a scratch buffer for thin first layers; this variant never
 * does.  It needs no hq_handle either (creating one allocates).
 *
 * It computes exactly what hq_conv2d computes on its lowered path (patch matrix, then the
 * tensor-core kernel; 8-bit operands, K = kh*kw*cin <= 4096, any cin), with the patch matrix and
 * the padded weights in a fixed 8 MiB array that is part of the library's device image.  A request
 * needing more than 8 MiB (n*ho*wo * K rounded up to 32, plus cout * that) returns HQ_ERR_WORKSPACE;
 * use hq_conv2d or a smaller batch then.  It calls no cudaMalloc, cudaFree or allocating library
 * routine.  The first call on a device looks up the array's device address, the driver's
 * tensor-map encoders and the kernel's shared-memory limit; make that first call outside any
 * stream capture.  All calls on a device share the one array and it keeps the previous call's
 * contents: the call rewrites everything it later reads and clears its status word on `stream`,
 * but two calls whose GPU work overlaps (different streams, or graphs replayed concurrently) race on
 * the array and give undefined results - serialise them.  The current device is used; pointers follow
 * the rules of hq_conv2d.  The one-time set-up is guarded by a lock, so first calls may come from several
 * host threads.  An expired device-side wait is reported by hq_conv2d_noalloc_sync.
 */
hq_status hq_conv2d_noalloc(const hq_tensor* in, const hq_conv_desc* desc, hq_tensor* out, void* stream);

/* Wait for `stream` and return HQ_ERR_TIMEOUT if a kernel of the hq_conv2d_noalloc calls queued on it gave
 * up a bounded device-side wait (the outputs of that call are not valid then), HQ_OK otherwise.  Like the
 * call it serves it allocates nothing; the word it reads is cleared by the next hq_conv2d_noalloc. */
hq_status hq_conv2d_noalloc_sync(void* stream);

/* Choose the convolution path: 0 = automatic, 1 = CUDA cores only, 2 = tensor cores or fail (HQ_ERR_UNSUPPORTED
 * for a shape they do not take, HQ_ERR_WORKSPACE when scratch memory for a lowered form cannot be had), 3 = like 2 and
 * the tensor-core kernel's launch shapes are chosen by what the layer allows, not by its size (small test cases
 * then reach the shapes of large layers). */
hq_status hq_set_conv_path(hq_handle* h, int32_t path);

/* Order in which the tensor-core convolutions (pixel tiles) and hq_concat_requant (pixels) of this handle walk their
 * tensors: 0 = from the first output pixel to the last (default), 1 = from the last to the first.  The results are identical; the order only decides which
 * end of a large tensor is touched first, and with it what a layer finds in the L2 of what the call before it wrote
 * (a network chooses the order layer by layer itself and ignores this setting).  (No counterpart in the paper.) */
hq_status hq_set_tile_order(hq_handle* h, int32_t order);

/* Self-test of the bounded device-side waits: one thread waits on a barrier that nothing ever signals, for at
 * most `budget_ms` milliseconds (1..2000), then records the expiry in the handle's status word and returns, as
 * every wait inside the kernels does after its own budget.  The next hq_sync reports HQ_ERR_TIMEOUT; the
 * context stays usable.  Asynchronous on `stream`. */
hq_status hq_expire_wait_selftest(hq_handle* h, int32_t budget_ms, void* stream);

/* Bit-width selection by integer linear programming (Section 3.4, Eq. 5).  Every one of n_layers layers takes
 * one of two precisions (choice 0 or 1, e.g. INT4 or INT8); the summed perturbation
 *   sum_i omega[i][b_i]   is minimised subject to
 *   sum_i size[i][b_i] <= size_limit,  sum_i bops[i][b_i] <= bops_limit,  sum_i latency[i][b_i] <= latency_limit
 * (M_i, G_i = b_w b_a MAC_i and Q_i of the paper; latency is what was measured per layer on the target GPU).
 * HOST pointers: four arrays of n_layers x 2 int64 values, [layer][choice], every value in [0, 2^40], in units of
 * the caller's choice; a negative limit switches that constraint off.  choice_out[n_layers] receives an optimal
 * assignment (any one of them when several are optimal) and objective_out, if not NULL, its perturbation.
 * Exact (depth-first branch and bound with fractional-knapsack bounds); pure host code, no GPU work, no handle.
 * Returns HQ_ERR_INFEASIBLE when no assignment meets the limits (choice_out untouched), HQ_ERR_INVALID_ARG for
 * NULL arrays, n_layers outside [0, 4096] or values out of range, HQ_ERR_UNSUPPORTED if the search exceeds
 * 2 * 10^8 nodes. */
hq_status hq_ilp_solve(int32_t n_layers, const int64_t* omega, const int64_t* size, const int64_t* bops,
                       const int64_t* latency, int64_t size_limit, int64_t bops_limit, int64_t latency_limit,
                       int32_t* choice_out, int64_t* objective_out);

const char* hq_status_string(hq_status s);

#ifdef __cplusplus
}
#endif
#endif /* HQ_H_ */
