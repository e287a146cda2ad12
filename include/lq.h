/*
 * lq.h - C ABI of the B200 (sm_100a) implementation of the LoRaQ fully quantized linear layer
 *
 *     Y = deq( Q4(X) * Q4(W - L1 L2) )  +  deq( Qb( Qb(X) * Qb(L1) ) * Qb(L2) )
 *
 * Notation follows the paper (Section 3.1): X in R^{m x d} activations, W in R^{d x n} weights,
 * Y = X W.  Here M = m rows (tokens x batch), K = d input features, N = n output features,
 * r = the rank of the low-rank branch, G = ceil(K / group) blocks of the 4-bit main format.
 *
 * Two main formats (Appendix A.3, Table 2), chosen by lq_config.group:
 *   group = 64  SINT4: signed 4-bit codes in [-7, 7], one fp16 scale per block of 64 along K;
 *               the per-block scale products are applied by the GEMM's epilogue warps.
 *   group = 32  MXINT4: the same codes, one power-of-two scale 2^e per block of 32 along K,
 *               e the smallest integer with 7 * 2^e >= max|v| of the block (the paper does not
 *               spell the rule out; this one never clips); the scales are applied by the tensor
 *               core itself (block-scaled MMA).  Every branch format; with the fp16 reference branch the
 *               tensor core also adds the branch product onto the same accumulator.
 *
 * Every function returns an lq_status; nothing throws, aborts or prints.  "host" / "device"
 * in a parameter comment says which address space the pointer lives in.  Device pointers and
 * the stream belong to the caller (e.g. a torch tensor's data_ptr() and a torch stream's
 * cuda_stream); everything behind lq_layer* / lq_act* is allocated and owned by the library
 * and released by the matching _free call.  Calls that take a stream are asynchronous on it.
 * There is no CPU fallback: without a CUDA device the device-side calls return LQ_ERR_CUDA.
 */
#ifndef LQ_H_
#define LQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LQ_OK = 0,
  LQ_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, handle/shape mismatch          */
  LQ_ERR_UNSUPPORTED = 2, /* a size or format outside what the kernels are built for         */
  LQ_ERR_ALLOC = 3,       /* host or device allocation failed                                 */
  LQ_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed (or no device)                 */
  LQ_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired (see lq_get_device_status)    */
  LQ_ERR_NUMERIC = 6      /* non-finite value met where the method needs finite ones          */
} lq_status;

/* Precision of the low-rank branch: bits of the two factors (W) and of the activations that
 * enter it, incl. the rank-r intermediate (A).  Section 3.3 quantizes the branch with an
 * operator Q2; the integer per-token / per-channel variants are this build's configurations. */
typedef enum {
  LQ_BRANCH_NONE = 0,   /* rank 0: plain W4A4                                  */
  LQ_BRANCH_W16A16 = 1, /* fp16 factors, fp16 activations (reference variant)  */
  LQ_BRANCH_W8A8 = 2,
  LQ_BRANCH_W6A6 = 3,
  LQ_BRANCH_W4A8 = 4,
  /* MX branches of the mixed-precision study (Section 4.3, Tables 3-4; Appendix A.3 "MX Formats"): factors in
   * blocks of 32 with a power-of-two scale and e4m3 / e2m3 / e2m1 elements; the activations of BOTH branches and
   * the rank-r intermediate are MXFP8e4.  Only with main_fmt = LQ_MAIN_MXFP4. */
  LQ_BRANCH_MXFP8 = 5,
  LQ_BRANCH_MXFP6 = 6,
  LQ_BRANCH_MXFP4 = 7,
  /* Integer MX branches of the same study (Table 3's integer rows): factors in blocks of 32 with a power-of-two
   * scale and signed 8-bit / 4-bit integer codes; the activations of BOTH branches and the rank-r intermediate
   * are MXINT8.  Only with main_fmt = LQ_MAIN_MXINT4_A8; rank <= 64 with MXINT8 factors, <= 128 with MXINT4 factors. */
  LQ_BRANCH_MXINT8 = 8,
  LQ_BRANCH_MXINT4 = 9
} lq_branch_fmt;

/* 4-bit format of the residual (main) branch, Appendix A.3. */
typedef enum {
  LQ_MAIN_AUTO = 0,    /* from `group`: 64 -> SINT4 (integer codes, fp16 scale per 64), 32 -> MXINT4           */
  LQ_MAIN_MXFP4 = 2,   /* MXFP4e2 weights (e2m1 elements, power-of-two scale per 32; group must be 32) times
                          MXFP8e4 activations, all scales applied by the tensor core (Tables 3-4)              */
  LQ_MAIN_MXINT4_A8 = 3 /* MXINT4 weights (group must be 32) times MXINT8 activations (Table 3's integer rows): an
                          8-bit code travels as two 4-bit digits, code = 16 hi + lo, each an exact E4M3 operand
                          with block scales 2^(e+4) and 2^e, so the tensor core applies every scale here too    */
} lq_main_fmt;

/* Element format of the activations (X for both branches, and the rank-r intermediate) of an MXFP layer.  The rank
 * study of Section 4.3 (Table 4) gives activations and factors ONE sub-16-bit format: MXFP8e4, or MXFP6e2. */
typedef enum {
  LQ_ACT_DEFAULT = 0,  /* SINT4 / MXINT4 main formats: their own 4-bit activations; MXFP4: MXFP8e4; MXINT4_A8: MXINT8 */
  LQ_ACT_MXFP6 = 6     /* MXFP6e2 activations; only with main_fmt = LQ_MAIN_MXFP4 (the weights' kernels do not change:
                          every e2m3 value is an e4m3 value)                                                     */
} lq_act_fmt;

typedef enum { LQ_OUT_F16 = 0, LQ_OUT_F32 = 1 } lq_out_dtype;

/* One layer's shape and calibration settings. */
typedef struct {
  int32_t K, N, rank; /* d, n and rho of Sections 3.1-3.2; rank in [0, 128]; K and N multiples of 8,
                         K <= 8192 (anything else: LQ_ERR_UNSUPPORTED)                              */
  int32_t group;      /* 64 = SINT4 (default), 32 = MXINT4: block length of the 4-bit main format  */
  int32_t branch;     /* an lq_branch_fmt                                                         */
  int32_t steps;      /* Adam steps on (L, R); 1000 in Appendix A "Optimization"                  */
  float lr;           /* 1e-4 for integer formats (Appendix A)                                    */
  float beta1, beta2, eps; /* Adam moments / epsilon; the paper is silent: 0.9, 0.999, 1e-8       */
  int32_t rot_steps;  /* steps of the rotation-aware optimisation of Section 3.3; 0 (default) = none,  */
  float rot_lr;       /* 500 steps at 0.5 (0.1 for the mixed-precision study) in Appendix A           */
  uint64_t seed;      /* start vectors of the host SVD iteration                                  */
  int32_t main_fmt;   /* an lq_main_fmt; 0 (default) = SINT4 / MXINT4 as `group` says                */
  int32_t act_fmt;    /* an lq_act_fmt; 0 (default) = the main format's own activations                 */
} lq_config;

typedef struct lq_layer lq_layer; /* opaque: Q1(P) codes+scales, Q2(L1), Q2(L2), bias (Figure 1)  */
typedef struct lq_act lq_act;     /* opaque: device buffers holding one batch of quantized
                                     activations for one layer shape (qx, sx, qb, sXb, tq, sT)   */

/* Fill *cfg with the defaults above for the given shape. */
lq_status lq_config_default(lq_config* cfg, int32_t K, int32_t N, int32_t rank, int32_t branch);

/* Data-free calibration of one weight, entirely on the host (Sections 3.2-3.3, Appendix A,
 * Appendix B.2): SVD initialisation L = -L0, R = R0; Adam on
 * mean((Q1(W + L R) - W - L R)^2) with the quantizer's derivative taken as zero; the best
 * iterate is kept; with cfg->rot_steps > 0 an orthogonal rotation Om of the factors (L1 Om,
 * Om^T L2: the same product) is then optimised to lower Q2's error (Cayley retraction steps,
 * best iterate kept); the factors are quantized with Q2; P = W - Q2(L1) Q2(L2) is quantized
 * with Q1 (SINT4 or MXINT4 blocks along K per output column, as cfg->group says; MXINT4 weight
 * exponents are kept within [-24, 15] so that 2^e is a finite fp16 number).  With main_fmt = LQ_MAIN_MXFP4,
 * Q1 is MXFP4e2 and Q2 the branch's MXFP format (blocks of 32 along each factor's contraction axis; exponent
 * floor(log2 max) - emax as in the OCP Microscaling conversion the paper cites; no rotation step: rot_steps must be 0).
 * With main_fmt = LQ_MAIN_MXINT4_A8, Q1 is MXINT4 and Q2 the branch's MX integer format (blocks of 32 along each
 * factor's contraction axis, the smallest power-of-two scale that does not clip; rot_steps must be 0).
 *   W_f16_host     [K][N] row-major IEEE half bits (the paper's d x n orientation), host
 *   bias_f16_host  [N] half bits or NULL, host
 *   out            receives a new layer (host copy only; see lq_layer_to_device)
 *   objective_trace[steps + 1] doubles or NULL, host: objective at every iterate, [0] = init
 * Errors: INVALID_ARG (null / bad shape), UNSUPPORTED (group not 64 or 32, ...),
 * NUMERIC (non-finite W), ALLOC. */
lq_status lq_calibrate(const lq_config* cfg, const uint16_t* W_f16_host,
                       const uint16_t* bias_f16_host, lq_layer** out, double* objective_trace);

/* Build a layer from already quantized parts (all host pointers, copied):
 *   Wq_packed [K][N/2] bytes: codes in [-7,7] as two's-complement nibbles, column 2j in the
 *             low nibble, column 2j+1 in the high nibble
 *   sw        [G][N] half bits: scale of block g of output column n (MXINT4: an exact power of
 *             two 2^e with e in [-24, 15], anything else is INVALID_ARG)
 *   L1, L2    integer branches: int8 codes [K][rank] and [rank][N]; W16A16: half bits, same shapes
 *   sL1, sL2  fp32 per-column scales [rank] and [N]; NULL for W16A16
 *   bias      [N] half bits or NULL
 * With rank == 0 or LQ_BRANCH_NONE the branch pointers are ignored.
 * MXFP layers (main_fmt = LQ_MAIN_MXFP4):
 *   Wq_packed [K][N/2] bytes: e2m1 bit patterns (sign, two exponent bits, one mantissa bit) as nibbles, same order
 *   sw        [ceil(K/32)][N] half bits: the block's power-of-two scale 2^e, e in [-24, 15]
 *   L1, L2    [K][rank] and [rank][N] bytes: e4m3 bit patterns of the elements (every e2m3 and e2m1 value is an
 *             e4m3 value, so the three MXFP branch formats arrive in one encoding)
 *   sL1, sL2  fp32 powers of two: [ceil(K/32)][rank] (blocks of L1 along K) and [ceil(rank/32)][N] (of L2 along rank)
 * Integer MX layers with 8-bit activations (main_fmt = LQ_MAIN_MXINT4_A8): Wq_packed and sw as for MXINT4;
 *   L1, L2    int8 codes [K][rank] and [rank][N], within [-127, 127] (LQ_BRANCH_MXINT8) or [-7, 7] (LQ_BRANCH_MXINT4)
 *   sL1, sL2  fp32 powers of two 2^e, e in [-120, 120]: [ceil(K/32)][rank] and [ceil(rank/32)][N] */
lq_status lq_layer_import(const lq_config* cfg, const uint8_t* Wq_packed, const uint16_t* sw,
                          const void* L1, const float* sL1, const void* L2, const float* sL2,
                          const uint16_t* bias, lq_layer** out);

/* Copy a layer's parts out into caller-sized host buffers (same layouts as lq_layer_import;
 * any pointer may be NULL to skip that part). */
lq_status lq_layer_export(const lq_layer* layer, uint8_t* Wq_packed, uint16_t* sw, void* L1,
                          float* sL1, void* L2, float* sL2, uint16_t* bias);

/* Shape of a layer handle. */
lq_status lq_layer_info(const lq_layer* layer, lq_config* cfg_out);

/* Upload the layer to `device` in the kernels' operand layout (allocates device memory;
 * synchronous).  Must precede lq_act_create / lq_quantize_act / lq_linear_forward. */
lq_status lq_layer_to_device(lq_layer* layer, int device);

lq_status lq_layer_free(lq_layer* layer);

/* Allocate the activation record for up to M_max rows of `layer`'s shape on `device`. */
lq_status lq_act_create(const lq_layer* layer, int32_t M_max, int device, lq_act** out);
lq_status lq_act_free(lq_act* act);

/* Dynamic activation quantization fused with the branch's down-projection (Figure 1;
 * Appendix A.2 "Quantization": both the residual and the low-rank branch consume quantized X).
 * One read of X produces
 *   qx, sx   4-bit codes / scales per token and block along K (Appendix A.3): fp16 scales per
 *            block of 64 (SINT4) or one exponent byte per block of 32 (MXINT4)
 *   qb, sXb  per-token branch codes / fp32 scale
 *   tq, sT   per-token codes / scale of the rank-r intermediate T = deq(qb) deq(L1)
 *   X_f16_dev  [M][K] row-major half, device, 16-byte aligned
 *   M          1 <= M <= M_max of `out`
 * X must be finite: the kernel does not look for infinities or NaNs (a row that holds one gets an
 * undefined scale and codes; nothing is flagged).  LQ_ERR_NUMERIC is raised only by the host-side
 * calls, for non-finite weights or scales.
 * Asynchronous on `cuda_stream` (a cudaStream_t). */
lq_status lq_quantize_act(const lq_layer* layer, const void* X_f16_dev, int32_t M, lq_act* out,
                          void* cuda_stream);

/* Y = sum_g sx sw (qx_g Wq_g) + sT sL2 (tq L2q) + bias: the 4-bit main product per group on
 * the tensor cores, per-group scales and the branch's up-projection applied in one epilogue
 * (Figure 1; Section 3.3).  For an MXINT4 layer the tensor core applies sx sw itself and the
 * epilogue only adds the branch and the bias.
 *   act    result of lq_quantize_act for this layer
 *   Y_dev  [M][N] row-major, half or float per `dtype`, device, 16-byte aligned
 * Asynchronous on `cuda_stream`. */
lq_status lq_linear_forward(const lq_layer* layer, const lq_act* act, void* Y_dev,
                            lq_out_dtype dtype, void* cuda_stream);

/* Whole path from host memory: copies X to the device, runs lq_quantize_act and
 * lq_linear_forward, copies Y back and waits for it.  X_f16_host [M][K], Y_host [M][N].
 * Rows are independent, so for M >= 512 the call is pipelined over up to eight row chunks (of at
 * least 256 rows): one chunk
 * is computed on `cuda_stream` while the next travels host -> device and the previous one
 * device -> host on two internal copy streams (this needs pinned host memory to overlap;
 * pageable memory works but serialises).  Staging buffers, streams and events inside `act`
 * are created on the first call.  Afterwards `act` holds the codes of all M rows. */
lq_status lq_linear_forward_host(const lq_layer* layer, lq_act* act, const void* X_f16_host,
                                 int32_t M, void* Y_host, lq_out_dtype dtype, void* cuda_stream);

/* The same without the final wait: returns once everything is queued; Y_host is complete when
 * `cuda_stream` has been synchronised (the stream is made to wait for the last copy).  X_f16_host
 * and Y_host must be pinned and must stay valid until then.  Calls for different layers on
 * different streams (each with its own `act`) overlap their copies in both directions, which a
 * sequence of waiting calls cannot: one layer's output travels device -> host while the next
 * layer's input travels host -> device.  Figure 1's data flow; the paper has no counterpart for
 * the transport itself. */
lq_status lq_linear_forward_host_async(const lq_layer* layer, lq_act* act, const void* X_f16_host,
                                       int32_t M, void* Y_host, lq_out_dtype dtype, void* cuda_stream);

/* (The paper has no counterpart for this entry point; it exists for deployment.)
 * Same result as lq_quantize_act followed by lq_linear_forward, for callers that may not
 * allocate device memory when they call: servers whose own pool owns all device memory once
 * start-up is over, loops with a fixed memory budget, plugins inside a framework that owns the
 * allocator - a raw allocation there can fail, fragment the pool, and stalls every stream while
 * it synchronises the device.  This call performs no allocation (no cudaMalloc / cudaFree,
 * no allocating library routine): the activation record lives in one fixed device array of
 * LQ_STATIC_SCRATCH_BYTES that is part of the library image, so every GPU that loads the
 * library holds that much memory until the process exits.  The caller passes only inputs and
 * outputs:
 *   layer      uploaded with lq_layer_to_device (that earlier call is where the layer's
 *              own device memory was allocated)
 *   X_f16_dev  [M][K] row-major half, device, 16-byte aligned
 *   Y_dev      [M][N] row-major half or float per `dtype`, device, 16-byte aligned
 * Limit: with Mp = M rounded up to 128, Kp = K rounded up to 128 and G2 = Kp / 64, the record
 * needs about 2*Mp*Kp + 4*G2*Mp + 136*Mp bytes (each part rounded up to 256); if that exceeds
 * LQ_STATIC_SCRATCH_BYTES - or if the layer's main format is MXINT4, which this entry point
 * does not cover - the call returns LQ_ERR_UNSUPPORTED and launches nothing
 * (8 MiB holds e.g. M = 256 at any supported K, or M = 1024 at K = 2240).
 * The first call on each device looks up the array's device address (one-time set-up, done
 * with that device current); make that first call before starting any stream capture.
 * All calls share the one array, which keeps the previous call's contents: each call first
 * clears the part it uses (on `cuda_stream`), and two calls that overlap on the GPU - other
 * streams, other threads - race on it; serialise them.  Asynchronous on `cuda_stream`. */
#define LQ_STATIC_SCRATCH_BYTES (8u << 20)
lq_status lq_linear_forward_static(const lq_layer* layer, const void* X_f16_dev, int32_t M, void* Y_dev,
                                   lq_out_dtype dtype, void* cuda_stream);

/* Decode the activation record of the last lq_quantize_act into plain host arrays (for
 * parity checks); NULL skips a part.  qx int8 [M][K], sx half bits [M][G] (MXINT4: the block
 * exponents e as int16 [M][G], since 2^e may lie below the fp16 range), qb int8 [M][K],
 * sXb float [M], tq int8 [M][rank] (W16A16: half bits [M][rank]), sT float [M].
 * MXFP: qx and tq are the e4m3 bytes, sT the block exponents of the intermediate as floats [M][ceil(rank/32)].
 * Integer MX with 8-bit activations: qx and tq are the int8 codes (16 hi + lo of the two stored digits), sx the
 * block exponents as for MXINT4, sT the block exponents of the intermediate as floats [M][ceil(rank/32)].
 * Synchronises `cuda_stream`. */
lq_status lq_act_export(const lq_act* act, int8_t* qx, uint16_t* sx, int8_t* qb, float* sXb,
                        void* tq, float* sT, void* cuda_stream);

/* Status word the kernels write when a bounded wait expires: code is an lq_status
 * (LQ_OK if none), stage identifies the waiting role.  Reading clears it.  Synchronises
 * the device. */
lq_status lq_get_device_status(int device, int32_t* code, int32_t* stage);

/* Self-test of the kernels' failure detection (the paper has no counterpart).  Every wait inside the
 * kernels is bounded: a role that waits longer than its limit records LQ_ERR_TIMEOUT and its
 * stage in the status word, and the kernel returns instead of hanging.  This call launches a
 * one-warp kernel that waits, with a limit of about 0.1 s, on a barrier that nothing ever arrives
 * on; afterwards lq_get_device_status must report {LQ_ERR_TIMEOUT, 4} and the device stays usable.
 * Asynchronous on `cuda_stream`. */
lq_status lq_selftest_wait_timeout(int device, void* cuda_stream);

/* Process-wide switches, read when a call is made; they are plain globals, so set them while no other
 * thread is inside the library (distinct handles may otherwise be used from distinct threads).
 *   "store_qb"     1: lq_quantize_act also writes the branch activation codes to HBM so that lq_act_export can
 *                  return them (parity tests); 0 (default): they stay on chip
 *   "gemm_ctas"    CTAs of the GEMM kernels; 0 (default) = one per SM
 *   "quant_ctas", "quant_warps"   residency and consumer warps of the quantizer kernel; 0 = chosen by the library
 *   "overlap"      1 (default): kernels are launched with programmatic stream serialization - a kernel's CTAs may take
 *                  their SMs and set up while the previous kernel on the stream drains, and wait (in the kernel) for
 *                  that kernel's completion before touching global memory; 0: plain launches
 *   "main_kind"    byte format that carries the 4-bit codes into the tensor cores; only 1 (E4M3) exists
 * Returns INVALID_ARG for an unknown name or value. */
lq_status lq_set_option(const char* name, int32_t value);

const char* lq_status_string(lq_status s);
/* Text of the last CUDA runtime error this host thread met inside the library ("no error" if none);
 * what LQ_ERR_CUDA stood for. */
const char* lq_last_cuda_error(void);
int lq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LQ_H_ */
