// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "lq.h"

#define LQ_GROUP 64
#define LQ_MX_BLOCK 32          // MXINT4: blocks of 32 with a power-of-two (E8M0) scale
#define LQ_BM 128            // rows per output tile (one tcgen05 MMA, M = 128)
#define LQ_BN 128            // columns per output tile
#define LQ_KSTAGE 128        // bytes of K per shared-memory stage row (two groups of 64 codes)
#define LQ_RCONT 128         // bytes per row of the branch containers (tq, L2q): rank <= 128
#define LQ_MAX_K 8192
#define LQ_MAX_RANK 128
#define LQ_HOST_CHUNKS 8       // row chunks (at most) lq_linear_forward_host overlaps (copy in / compute / copy out)

// role identifiers reported through the device status word
enum { LQ_STAGE_NONE = 0, LQ_STAGE_PRODUCER = 1, LQ_STAGE_MMA = 2, LQ_STAGE_DRAIN = 3, LQ_STAGE_TEARDOWN = 4, LQ_STAGE_QUANT = 5 };

enum { LQ_KIND_I8 = 0, LQ_KIND_E4M3 = 1 };

static inline int lq_ceil_div(int a, int b) { return (a + b - 1) / b; }
static inline int lq_round_up(int a, int b) { return lq_ceil_div(a, b) * b; }

// offset of the scale byte of row (or column) i and 32-block kb inside its [tile][kb/4] chunk of 512 bytes
static inline size_t lq_sf_offset(int i, int kb, int Kpad) {
  return ((size_t)(i / 128) * (Kpad / 128) + kb / 4) * 512 + 16 * (i % 32) + 4 * ((i % 128) / 32) + kb % 4;
}

// the same for the weight scales, whose chunks are ordered [kb/4][tile] so that neighbouring column tiles are contiguous
static inline size_t lq_sfb_offset(int n, int kb, int Npad) {
  return ((size_t)(kb / 4) * (Npad / 128) + n / 128) * 512 + 16 * (n % 32) + 4 * ((n % 128) / 32) + kb % 4;
}

static inline bool lq_branch_is_mxfp(int branch) {
  return branch == LQ_BRANCH_MXFP8 || branch == LQ_BRANCH_MXFP6 || branch == LQ_BRANCH_MXFP4;
}
// An 8-bit code c in [-127, 127] as two digits, c = 16 hi + lo with lo in [-8, 7] and hi in [-8, 8]: both are exact
// E4M3 values, so a block-scaled MMA can carry an 8-bit integer operand as two planes with scales 2^(e+4) and 2^e.
static inline void lq_split_digits(int c, int* hi, int* lo) {
  const int l = ((c + 8) & 15) - 8;
  *lo = l; *hi = (c - l) / 16;
}
// E4M3 byte of an integer in [-8, 8] (bias 7, three mantissa bits; 8 = 1.0 * 2^3)
static inline uint8_t lq_digit_e4m3(int d) {
  static const uint8_t mag[9] = {0x00, 0x38, 0x40, 0x44, 0x48, 0x4A, 0x4C, 0x4E, 0x50};
  return (uint8_t)((d < 0 ? 0x80 : 0x00) | mag[d < 0 ? -d : d]);
}
static inline bool lq_branch_is_mxint(int branch) { return branch == LQ_BRANCH_MXINT8 || branch == LQ_BRANCH_MXINT4; }
static inline int lq_branch_wbits(int branch) {
  return branch == LQ_BRANCH_W8A8 ? 8 : branch == LQ_BRANCH_W6A6 ? 6 : branch == LQ_BRANCH_W4A8 ? 4 : 0;
}
static inline int lq_branch_abits(int branch) {
  return branch == LQ_BRANCH_W8A8 ? 8 : branch == LQ_BRANCH_W6A6 ? 6 : branch == LQ_BRANCH_W4A8 ? 8 : 0;
}

struct lq_layer {
  lq_config cfg;
  int K, N, r, G;          // logical sizes
  int Kpad, Npad, Gpad;    // Kpad: multiple of 128; Npad: multiple of LQ_BN; Gpad = Kpad / 64
  bool integer_branch, f16_branch, has_bias;
  bool mx;                     // MX main branch (cfg.group == 32): G counts blocks of 32, sw holds powers of two
  bool mxfp;                   // MXFP4 weights x MXFP8e4 activations (implies mx); the branch, if any, is MXFP too
  bool a8;                     // MXINT4 weights x MXINT8 activations (implies mx): 8-bit codes travel as two E4M3 digit
                               // planes (hi, lo); factors: int8 codes in L1q / L2q with block scales in s1b / s2b
  std::vector<uint8_t> Wq8h;   // mxfp: [K][N] e4m3 bytes of the e2m1 weight elements
  std::vector<uint8_t> L1e, L2e;   // mxfp: e4m3 bytes of the factor elements, [K][r] and [r][N]
  std::vector<float> s1b, s2b; // mxfp: block scales 2^e of L1 [ceil(K/32)][r] and of L2 [ceil(r/32)][N]
  // host copy, canonical layouts
  std::vector<int8_t> Wq;      // [K][N]
  std::vector<uint16_t> sw;    // [G][N] half bits
  std::vector<int8_t> L1q;     // [K][r]
  std::vector<int8_t> L2q;     // [r][N]
  std::vector<float> sL1, sL2; // [r], [N]
  std::vector<uint16_t> L1h;   // [K][r] half bits (W16A16)
  std::vector<uint16_t> L2h;   // [r][N]
  std::vector<uint16_t> bias;  // [N]
  // device copy, operand layouts
  int device;
  int main_kind;               // LQ_KIND_*: byte encoding of the 4-bit codes in the MMA operands
  uint8_t* d_Wq8;              // [Npad][Kpad] bytes, K contiguous (B operand, K-major)
  float* d_sw;                 // [Gpad][Npad] fp32 (exact images of the fp16 scales)
  uint8_t* d_L1f;              // [Kpad/64][r tiles][32 lanes][16 bytes]: first factor in mma.sync B-fragment order (integer
                               // branches): lane 4 c + t holds k = 64 box + 16 t + 0..15 of column 8 tile + c
  uint16_t* d_L1h;             // the same order with 16 halves per lane (W16A16)
  float* d_sL1;                // [LQ_MAX_RANK]
  uint8_t* d_L2c;              // [Npad][LQ_RCONT] bytes: int8 codes (or up to 64 halves) of column n, r contiguous
  float* d_sL2;                // [Npad]  (ones for W16A16)
  float* d_bias;               // [Npad]  (zeros without bias)
  float* d_s1b;                // mxfp: 2^e1 [Kpad/32][rpad] (zero-padded columns)
  uint8_t* d_sfl2;             // mxfp: E8M0 bytes of L2's block scales, [1][Npad/128][512] in the tensor-memory layout
  uint8_t* d_sfb;              // MXINT4: E8M0 bytes of the weight scales, [Kpad/128][Npad/128][512] in the 32 x 16-byte
                               // layout tensor memory wants (byte 16*(n%32) + 4*((n%128)/32) + block%4)
  CUtensorMap tmB;             // over d_Wq8, box [LQ_BN][128B], 128B swizzle
  CUtensorMap tmB2;            // over d_Wq8, box [2 LQ_BN][128B]: both halves of a 256-column tile in one copy
  CUtensorMap tmL2;            // over d_L2c, box [LQ_BN][128B], 128B swizzle
};

struct lq_act {
  int K, N, r, G, Kpad, Gpad, branch;
  bool mx, mxfp, a8;
  int planes;                  // 1, or 2 (a8): digit planes of the main codes; qx8 rows are planes * Kpad bytes
  int tq_stride;               // bytes per row of d_tq: LQ_RCONT, or 2 LQ_RCONT when the intermediate's two digit planes get a
                               // container each (a8 with MXINT4 factors: rank up to 128), d_sft then holds two chunks per row block
  uint8_t* d_sft;              // mxfp: E8M0 bytes of the rank-r intermediate's block scales, [Mpad/128][1][512]
  uint8_t* d_sfa;              // MX: E8M0 bytes of the activation scales, [Mpad/128][Kpad/128][512], same layout
  int M_max, Mpad, device, main_kind;
  int M;                       // rows of the last lq_quantize_act
  uint8_t* d_qx8;              // [Mpad][Kpad] operand bytes of the 4-bit codes (A operand, K-major)
  float* d_sx;                 // [Gpad][Mpad] fp32 images of the fp16 scales
  int8_t* d_qb;                // [Mpad][Kpad] branch activation codes
  float* d_sXb;                // [Mpad]
  uint8_t* d_tq;               // [Mpad][LQ_RCONT] bytes: int8 codes (or halves) of T, r contiguous
  float* d_sT;                 // [Mpad] (ones for W16A16)
  void* d_Xstage;              // lazily allocated staging for lq_linear_forward_host
  void* d_Ystage;
  size_t ystage_bytes;
  cudaStream_t s_h2d, s_d2h;   // copy streams of lq_linear_forward_host's row-chunk pipeline (created on first use)
  cudaEvent_t ev_x[LQ_HOST_CHUNKS], ev_y[LQ_HOST_CHUNKS], ev_begin, ev_end;
  bool pipe_ready;
  CUtensorMap tmA;             // over d_qx8, box [LQ_BM][128B], 128B swizzle
  CUtensorMap tmT;             // over d_tq,  box [LQ_BM][128B], 128B swizzle
};

// remembers the last failing CUDA runtime code (per host thread) for lq_last_cuda_error(); returns its argument
cudaError_t lq_note_cuda(cudaError_t e);

// device status word (one per device, allocated on first use): {code, stage}
int32_t* lq_device_status_ptr(int device);

// kernels' host launchers (defined in lq_quant.cu / lq_gemm.cu)
lq_status lq_launch_quantize(const lq_layer* L, const void* X, int M, lq_act* A, cudaStream_t st);
lq_status lq_launch_gemm(const lq_layer* L, const lq_act* A, void* Y, lq_out_dtype dt, cudaStream_t st);
lq_status lq_gemm_prepare(int device);
lq_status lq_launch_gemm_mx(const lq_layer* L, const lq_act* A, void* Y, lq_out_dtype dt, cudaStream_t st);
lq_status lq_gemm_mx_prepare(int device);
lq_status lq_launch_wait_probe(int device, cudaStream_t st);   // bounded-wait self-test kernel
int lq_quant_rank_tiles(int r, bool f16);   // 8-column tiles of the rank the quantizer kernels are built for (2, 4, 8 or 16)

// TMA descriptors (lq_api.cu).  lq_make_tmap_bytes: 2-D byte tensor [rows][row_bytes], box [box_rows][128 bytes],
// 128-byte swizzle.  lq_make_tmap_rows16: fp16 activations [M][K], box 16 rows x 64 values, 128-byte swizzle,
// zeros outside the tensor.
lq_status lq_make_tmap_bytes(CUtensorMap* tm, void* base, uint64_t rows, uint64_t row_bytes, uint32_t box_rows);
lq_status lq_make_tmap_rows16(CUtensorMap* tm, const void* X, uint64_t M, uint64_t K);

// byte an MMA operand carries for a 4-bit code q in [-7, 7]
static inline uint8_t lq_encode_code_host(int q, int kind) {
  if (kind == LQ_KIND_I8) return (uint8_t)(int8_t)q;
  static const uint8_t mag[8] = {0x00, 0x38, 0x40, 0x44, 0x48, 0x4A, 0x4C, 0x4E};  // E4M3 of 0..7
  int a = q < 0 ? -q : q;
  return (uint8_t)(mag[a] | (q < 0 ? 0x80 : 0));
}

extern int g_lq_main_kind;   // option "main_kind"
extern int g_lq_gemm_ctas;   // option "gemm_ctas" (0 = one per SM)
extern int g_lq_quant_warps, g_lq_quant_ctas;   // options "quant_warps", "quant_ctas": 0 = chosen by the launcher
extern int g_lq_overlap;     // option "overlap": launch kernels with programmatic stream serialization
extern int g_lq_store_qb;    // option "store_qb": also write the branch activation codes to HBM (parity export)

#ifdef __CUDACC__
// Launches `kernel` on `st`.  With the "overlap" option the launch carries programmatic stream serialization: the
// kernel's CTAs may become resident and run their set-up (barriers, tensor memory) while the previous kernel on the
// stream is still draining its last tiles; every kernel of this library executes griddepcontrol.wait after that set-up,
// before it reads or writes global memory, and griddepcontrol.launch_dependents right before it, so that the chain
// quantizer -> GEMM -> next quantizer overlaps its launch gaps and tails.  All kernels here are persistent (the whole
// grid is resident at once), so a waiting successor never holds an SM that a predecessor CTA still needs.
template <typename... KArgs, typename... Args>
static inline cudaError_t lq_launch(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3((unsigned)grid); lc.blockDim = dim3((unsigned)block); lc.dynamicSmemBytes = smem; lc.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at; lc.numAttrs = g_lq_overlap ? 1 : 0;
  return cudaLaunchKernelEx(&lc, kernel, std::forward<Args>(args)...);
}
#endif
