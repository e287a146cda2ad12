// Handles, import/export, device upload and the host-side plumbing of the C ABI.
#include <cuda_fp16.h>
#include <math.h>
#include <string.h>

#include <mutex>
#include <new>

#include "lq_internal.h"

int g_lq_main_kind = LQ_KIND_E4M3;
int g_lq_gemm_ctas = 0;
int g_lq_store_qb = 0;
int g_lq_quant_warps = 0;
int g_lq_quant_ctas = 0;
int g_lq_overlap = 1;

static thread_local cudaError_t t_last_cuda_error = cudaSuccess;

cudaError_t lq_note_cuda(cudaError_t e) {
  if (e != cudaSuccess) t_last_cuda_error = e;
  return e;
}

extern "C" const char* lq_last_cuda_error(void) { return cudaGetErrorString(t_last_cuda_error); }

#define CUDA_OK(expr)                                      \
  do {                                                     \
    if (lq_note_cuda(expr) != cudaSuccess) return LQ_ERR_CUDA; \
  } while (0)

static inline float h2f(uint16_t h) {
  __half_raw r; r.x = h;
  return __half2float(__half(r));
}

extern "C" const char* lq_status_string(lq_status s) {
  switch (s) {
    case LQ_OK: return "ok";
    case LQ_ERR_INVALID_ARG: return "invalid argument";
    case LQ_ERR_UNSUPPORTED: return "unsupported size or format";
    case LQ_ERR_ALLOC: return "allocation failed";
    case LQ_ERR_CUDA: return "CUDA call failed";
    case LQ_ERR_TIMEOUT: return "bounded device wait expired";
    case LQ_ERR_NUMERIC: return "non-finite value";
  }
  return "unknown status";
}

extern "C" int lq_version(void) { return 100; }

extern "C" lq_status lq_set_option(const char* name, int32_t value) {
  if (!name) return LQ_ERR_INVALID_ARG;
  if (!strcmp(name, "main_kind")) {
    if (value != LQ_KIND_E4M3) return LQ_ERR_INVALID_ARG;   // the only operand format the kernels are built for
    g_lq_main_kind = value;
    return LQ_OK;
  }
  if (!strcmp(name, "store_qb")) {
    g_lq_store_qb = value != 0;
    return LQ_OK;
  }
  if (!strcmp(name, "quant_warps")) {
    if (value < 0 || value > 9) return LQ_ERR_INVALID_ARG;
    g_lq_quant_warps = value;
    return LQ_OK;
  }
  if (!strcmp(name, "quant_ctas")) {
    if (value < 0 || value > 4) return LQ_ERR_INVALID_ARG;
    g_lq_quant_ctas = value;
    return LQ_OK;
  }
  if (!strcmp(name, "overlap")) {
    if (value != 0 && value != 1) return LQ_ERR_INVALID_ARG;
    g_lq_overlap = value;
    return LQ_OK;
  }
  if (!strcmp(name, "gemm_ctas")) {
    if (value < 0) return LQ_ERR_INVALID_ARG;
    g_lq_gemm_ctas = value;
    return LQ_OK;
  }
  return LQ_ERR_INVALID_ARG;
}

extern "C" lq_status lq_config_default(lq_config* cfg, int32_t K, int32_t N, int32_t rank, int32_t branch) {
  if (!cfg) return LQ_ERR_INVALID_ARG;
  memset(cfg, 0, sizeof(*cfg));
  cfg->K = K; cfg->N = N; cfg->rank = rank; cfg->group = LQ_GROUP; cfg->branch = branch;
  cfg->steps = 1000; cfg->lr = 1e-4f; cfg->beta1 = 0.9f; cfg->beta2 = 0.999f; cfg->eps = 1e-8f;
  cfg->rot_steps = 0; cfg->rot_lr = 0.5f; cfg->seed = 0;
  cfg->main_fmt = LQ_MAIN_AUTO; cfg->act_fmt = LQ_ACT_DEFAULT;
  if (lq_branch_is_mxfp(branch)) { cfg->main_fmt = LQ_MAIN_MXFP4; cfg->group = LQ_MX_BLOCK; cfg->lr = 1e-3f; }
  if (lq_branch_is_mxint(branch)) { cfg->main_fmt = LQ_MAIN_MXINT4_A8; cfg->group = LQ_MX_BLOCK; }
  return LQ_OK;
}

static lq_status check_config(const lq_config* c) {
  if (!c) return LQ_ERR_INVALID_ARG;
  if (c->K <= 0 || c->N <= 0 || c->rank < 0) return LQ_ERR_INVALID_ARG;
  if (c->branch < LQ_BRANCH_NONE || c->branch > LQ_BRANCH_MXINT4) return LQ_ERR_INVALID_ARG;
  if (c->group != LQ_GROUP && c->group != LQ_MX_BLOCK) return LQ_ERR_UNSUPPORTED;
  if (c->main_fmt != LQ_MAIN_AUTO && c->main_fmt != LQ_MAIN_MXFP4 && c->main_fmt != LQ_MAIN_MXINT4_A8) return LQ_ERR_INVALID_ARG;
  // MXFP4 weights go with blocks of 32 and an MXFP (or no) branch; MXFP branches go with nothing else
  if (c->main_fmt == LQ_MAIN_MXFP4 && (c->group != LQ_MX_BLOCK || !(c->branch == LQ_BRANCH_NONE || lq_branch_is_mxfp(c->branch))))
    return LQ_ERR_UNSUPPORTED;
  if (c->main_fmt != LQ_MAIN_MXFP4 && lq_branch_is_mxfp(c->branch)) return LQ_ERR_UNSUPPORTED;
  if (c->act_fmt != LQ_ACT_DEFAULT && !(c->act_fmt == LQ_ACT_MXFP6 && c->main_fmt == LQ_MAIN_MXFP4)) return LQ_ERR_UNSUPPORTED;
  // MXINT8 activations go with MXINT4 weights in blocks of 32 and an integer MX (or no) branch; MXINT8 factors: rank <= 64
  // (both operands of the up-projection carry two digit planes, which share a 128-byte container each); MXINT4 factors:
  // rank <= 128 (one plane for L2, a container per plane for the intermediate)
  if (c->main_fmt == LQ_MAIN_MXINT4_A8 &&
      (c->group != LQ_MX_BLOCK || !(c->branch == LQ_BRANCH_NONE || lq_branch_is_mxint(c->branch)) || (c->branch == LQ_BRANCH_MXINT8 && c->rank > 64)))
    return LQ_ERR_UNSUPPORTED;
  if (c->main_fmt != LQ_MAIN_MXINT4_A8 && lq_branch_is_mxint(c->branch)) return LQ_ERR_UNSUPPORTED;
  if (c->K > LQ_MAX_K || (c->K % 8) != 0) return LQ_ERR_UNSUPPORTED;
  if ((c->N % 8) != 0) return LQ_ERR_UNSUPPORTED;
  if (c->rank > LQ_MAX_RANK) return LQ_ERR_UNSUPPORTED;
  if (c->branch == LQ_BRANCH_W16A16 && c->rank > 64) return LQ_ERR_UNSUPPORTED;
  if (c->rot_steps < 0) return LQ_ERR_INVALID_ARG;
  return LQ_OK;
}

// Shared by lq_layer_import and lq_calibrate: an empty layer with sizes filled in.
lq_layer* lq_layer_new(const lq_config* cfg) {
  lq_layer* L = new (std::nothrow) lq_layer();
  if (!L) return nullptr;
  L->cfg = *cfg;
  L->K = cfg->K; L->N = cfg->N;
  L->r = (cfg->branch == LQ_BRANCH_NONE) ? 0 : cfg->rank;
  if (L->r == 0) L->cfg.branch = LQ_BRANCH_NONE;
  L->cfg.rank = L->r;
  L->mx = cfg->group == LQ_MX_BLOCK;
  L->mxfp = cfg->main_fmt == LQ_MAIN_MXFP4;
  L->a8 = cfg->main_fmt == LQ_MAIN_MXINT4_A8;
  L->G = lq_ceil_div(L->K, cfg->group);
  L->Kpad = lq_round_up(L->K, LQ_KSTAGE);
  L->Gpad = L->Kpad / LQ_GROUP;
  L->Npad = lq_round_up(L->N, LQ_BN);
  L->integer_branch = L->r > 0 && L->cfg.branch != LQ_BRANCH_W16A16 && !lq_branch_is_mxfp(L->cfg.branch) && !lq_branch_is_mxint(L->cfg.branch);
  L->f16_branch = L->r > 0 && L->cfg.branch == LQ_BRANCH_W16A16;
  L->has_bias = false;
  L->device = -1;
  L->main_kind = g_lq_main_kind;
  L->d_Wq8 = nullptr; L->d_sw = nullptr; L->d_L1f = nullptr; L->d_L1h = nullptr; L->d_sL1 = nullptr;
  L->d_L2c = nullptr; L->d_sL2 = nullptr; L->d_bias = nullptr; L->d_sfb = nullptr;
  L->d_s1b = nullptr; L->d_sfl2 = nullptr;
  return L;
}

// e2m1 bit pattern (sign, two exponent bits, one mantissa bit) -> the e4m3 byte of the same value
static inline uint8_t e2m1_to_e4m3(int nib) {
  static const uint8_t mag[8] = {0x00, 0x30, 0x38, 0x3C, 0x40, 0x44, 0x48, 0x4C};   // 0, 0.5, 1, 1.5, 2, 3, 4, 6
  return (uint8_t)(mag[nib & 7] | ((nib & 8) ? 0x80 : 0));
}
static inline int e4m3_to_e2m1(uint8_t b) {
  static const uint8_t mag[8] = {0x00, 0x30, 0x38, 0x3C, 0x40, 0x44, 0x48, 0x4C};
  for (int i = 0; i < 8; ++i)
    if ((b & 0x7F) == mag[i]) return i | ((b & 0x80) ? 8 : 0);
  return -1;
}
// power of two held in a float -> its exponent (false if the value is not a positive power of two)
static inline bool pow2_exponent(float v, int* e) {
  int x = 0;
  if (!(v > 0.f) || !isfinite(v) || frexpf(v, &x) != 0.5f) return false;
  *e = x - 1;
  return true;
}

extern "C" lq_status lq_layer_import(const lq_config* cfg, const uint8_t* Wq_packed, const uint16_t* sw,
                                     const void* L1, const float* sL1, const void* L2, const float* sL2,
                                     const uint16_t* bias, lq_layer** out) {
  lq_status st = check_config(cfg);
  if (st != LQ_OK) return st;
  if (!Wq_packed || !sw || !out) return LQ_ERR_INVALID_ARG;
  lq_layer* L = lq_layer_new(cfg);
  if (!L) return LQ_ERR_ALLOC;
  const int K = L->K, N = L->N, r = L->r, G = L->G;
  if (r > 0 && (!L1 || !L2)) { delete L; return LQ_ERR_INVALID_ARG; }
  if (L->integer_branch && (!sL1 || !sL2)) { delete L; return LQ_ERR_INVALID_ARG; }
  if (L->mxfp) {
    const int nbK = lq_ceil_div(K, LQ_MX_BLOCK), nbR = lq_ceil_div(r > 0 ? r : 1, LQ_MX_BLOCK);
    if (r > 0 && (!sL1 || !sL2)) { delete L; return LQ_ERR_INVALID_ARG; }
    try {
      L->Wq8h.resize((size_t)K * N);
      for (int k = 0; k < K; ++k)
        for (int j = 0; j < N / 2; ++j) {
          const uint8_t b = Wq_packed[(size_t)k * (N / 2) + j];
          L->Wq8h[(size_t)k * N + 2 * j] = e2m1_to_e4m3(b & 0xF);
          L->Wq8h[(size_t)k * N + 2 * j + 1] = e2m1_to_e4m3(b >> 4);
        }
      L->sw.assign(sw, sw + (size_t)G * N);
      for (size_t i = 0; i < L->sw.size(); ++i) {
        int e = 0;
        if (!pow2_exponent(h2f(L->sw[i]), &e)) { delete L; return LQ_ERR_INVALID_ARG; }
      }
      if (r > 0) {
        const uint8_t* a = (const uint8_t*)L1; const uint8_t* b = (const uint8_t*)L2;
        L->L1e.assign(a, a + (size_t)K * r);
        L->L2e.assign(b, b + (size_t)r * N);
        for (uint8_t v : L->L1e) if ((v & 0x7F) == 0x7F) { delete L; return LQ_ERR_NUMERIC; }   // e4m3 NaN
        for (uint8_t v : L->L2e) if ((v & 0x7F) == 0x7F) { delete L; return LQ_ERR_NUMERIC; }
        L->s1b.assign(sL1, sL1 + (size_t)nbK * r);
        L->s2b.assign(sL2, sL2 + (size_t)nbR * N);
        int e = 0;
        for (float v : L->s1b) if (!pow2_exponent(v, &e)) { delete L; return LQ_ERR_INVALID_ARG; }
        for (float v : L->s2b) if (!pow2_exponent(v, &e) || e < -127 || e > 127) { delete L; return LQ_ERR_INVALID_ARG; }
      }
      if (bias) { L->bias.assign(bias, bias + N); L->has_bias = true; }
    } catch (const std::bad_alloc&) { delete L; return LQ_ERR_ALLOC; }
    *out = L;
    return LQ_OK;
  }
  try {
    L->Wq.resize((size_t)K * N);
    for (int k = 0; k < K; ++k)
      for (int j = 0; j < N / 2; ++j) {
        uint8_t b = Wq_packed[(size_t)k * (N / 2) + j];
        int lo = (int)(b & 0xF), hi = (int)(b >> 4);
        lo = lo >= 8 ? lo - 16 : lo; hi = hi >= 8 ? hi - 16 : hi;
        if (lo < -7 || hi < -7) { delete L; return LQ_ERR_INVALID_ARG; }
        L->Wq[(size_t)k * N + 2 * j] = (int8_t)lo;
        L->Wq[(size_t)k * N + 2 * j + 1] = (int8_t)hi;
      }
    L->sw.assign(sw, sw + (size_t)G * N);
    for (size_t i = 0; i < L->sw.size(); ++i) {
      const float v = h2f(L->sw[i]);
      if (!isfinite(v)) { delete L; return LQ_ERR_NUMERIC; }
      int x = 0;
      if (L->mx && !(v > 0.f && frexpf(v, &x) == 0.5f)) { delete L; return LQ_ERR_INVALID_ARG; }   // MXINT4 scales are powers of two
    }
    if (L->integer_branch) {
      const int qm = (1 << (lq_branch_wbits(L->cfg.branch) - 1)) - 1;
      const int8_t* a = (const int8_t*)L1; const int8_t* b = (const int8_t*)L2;
      L->L1q.assign(a, a + (size_t)K * r);
      L->L2q.assign(b, b + (size_t)r * N);
      for (int8_t v : L->L1q) if (v > qm || v < -qm) { delete L; return LQ_ERR_INVALID_ARG; }
      for (int8_t v : L->L2q) if (v > qm || v < -qm) { delete L; return LQ_ERR_INVALID_ARG; }
      L->sL1.assign(sL1, sL1 + r);
      L->sL2.assign(sL2, sL2 + N);
      for (float v : L->sL1) if (!isfinite(v)) { delete L; return LQ_ERR_NUMERIC; }
      for (float v : L->sL2) if (!isfinite(v)) { delete L; return LQ_ERR_NUMERIC; }
    } else if (L->f16_branch) {
      const uint16_t* a = (const uint16_t*)L1; const uint16_t* b = (const uint16_t*)L2;
      L->L1h.assign(a, a + (size_t)K * r);
      L->L2h.assign(b, b + (size_t)r * N);
    } else if (L->a8 && r > 0) {
      if (!sL1 || !sL2) { delete L; return LQ_ERR_INVALID_ARG; }
      const int qm = L->cfg.branch == LQ_BRANCH_MXINT8 ? 127 : 7;
      const int nbK = lq_ceil_div(K, LQ_MX_BLOCK), nbR = lq_ceil_div(r, LQ_MX_BLOCK);
      const int8_t* a = (const int8_t*)L1; const int8_t* b = (const int8_t*)L2;
      L->L1q.assign(a, a + (size_t)K * r);
      L->L2q.assign(b, b + (size_t)r * N);
      for (int8_t v : L->L1q) if (v > qm || v < -qm) { delete L; return LQ_ERR_INVALID_ARG; }
      for (int8_t v : L->L2q) if (v > qm || v < -qm) { delete L; return LQ_ERR_INVALID_ARG; }
      L->s1b.assign(sL1, sL1 + (size_t)nbK * r);
      L->s2b.assign(sL2, sL2 + (size_t)nbR * N);
      int e = 0;
      for (float v : L->s1b) if (!pow2_exponent(v, &e) || e < -120 || e > 120) { delete L; return LQ_ERR_INVALID_ARG; }
      for (float v : L->s2b) if (!pow2_exponent(v, &e) || e < -120 || e > 120) { delete L; return LQ_ERR_INVALID_ARG; }
    }
    if (bias) { L->bias.assign(bias, bias + N); L->has_bias = true; }
  } catch (const std::bad_alloc&) { delete L; return LQ_ERR_ALLOC; }
  *out = L;
  return LQ_OK;
}

extern "C" lq_status lq_layer_export(const lq_layer* L, uint8_t* Wq_packed, uint16_t* sw, void* L1,
                                     float* sL1, void* L2, float* sL2, uint16_t* bias) {
  if (!L) return LQ_ERR_INVALID_ARG;
  const int K = L->K, N = L->N, r = L->r;
  if (L->mxfp) {
    if (Wq_packed)
      for (int k = 0; k < K; ++k)
        for (int j = 0; j < N / 2; ++j)
          Wq_packed[(size_t)k * (N / 2) + j] = (uint8_t)(e4m3_to_e2m1(L->Wq8h[(size_t)k * N + 2 * j]) |
                                                         (e4m3_to_e2m1(L->Wq8h[(size_t)k * N + 2 * j + 1]) << 4));
    if (sw) memcpy(sw, L->sw.data(), L->sw.size() * sizeof(uint16_t));
    if (r > 0) {
      if (L1) memcpy(L1, L->L1e.data(), L->L1e.size());
      if (L2) memcpy(L2, L->L2e.data(), L->L2e.size());
      if (sL1) memcpy(sL1, L->s1b.data(), L->s1b.size() * sizeof(float));
      if (sL2) memcpy(sL2, L->s2b.data(), L->s2b.size() * sizeof(float));
    }
    if (bias && L->has_bias) memcpy(bias, L->bias.data(), N * sizeof(uint16_t));
    return LQ_OK;
  }
  if (Wq_packed)
    for (int k = 0; k < K; ++k)
      for (int j = 0; j < N / 2; ++j) {
        int lo = L->Wq[(size_t)k * N + 2 * j], hi = L->Wq[(size_t)k * N + 2 * j + 1];
        Wq_packed[(size_t)k * (N / 2) + j] = (uint8_t)((lo & 0xF) | ((hi & 0xF) << 4));
      }
  if (sw) memcpy(sw, L->sw.data(), L->sw.size() * sizeof(uint16_t));
  if (L->integer_branch) {
    if (L1) memcpy(L1, L->L1q.data(), (size_t)K * r);
    if (L2) memcpy(L2, L->L2q.data(), (size_t)r * N);
    if (sL1) memcpy(sL1, L->sL1.data(), r * sizeof(float));
    if (sL2) memcpy(sL2, L->sL2.data(), N * sizeof(float));
  } else if (L->f16_branch) {
    if (L1) memcpy(L1, L->L1h.data(), (size_t)K * r * 2);
    if (L2) memcpy(L2, L->L2h.data(), (size_t)r * N * 2);
  } else if (L->a8 && r > 0) {
    if (L1) memcpy(L1, L->L1q.data(), (size_t)K * r);
    if (L2) memcpy(L2, L->L2q.data(), (size_t)r * N);
    if (sL1) memcpy(sL1, L->s1b.data(), L->s1b.size() * sizeof(float));
    if (sL2) memcpy(sL2, L->s2b.data(), L->s2b.size() * sizeof(float));
  }
  if (bias && L->has_bias) memcpy(bias, L->bias.data(), N * sizeof(uint16_t));
  return LQ_OK;
}

extern "C" lq_status lq_layer_info(const lq_layer* L, lq_config* cfg_out) {
  if (!L || !cfg_out) return LQ_ERR_INVALID_ARG;
  *cfg_out = L->cfg;
  return LQ_OK;
}

// ---- TMA descriptors ---------------------------------------------------------------------
typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static encode_tiled_fn get_encode_fn() {
  static encode_tiled_fn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (encode_tiled_fn)p;
  });
  return fn;
}

// 2-D byte tensor [rows][row_bytes], box [box_rows][128 bytes], 128-byte swizzle.
lq_status lq_make_tmap_bytes(CUtensorMap* tm, void* base, uint64_t rows, uint64_t row_bytes, uint32_t box_rows) {
  encode_tiled_fn fn = get_encode_fn();
  if (!fn) return LQ_ERR_CUDA;
  cuuint64_t dims[2] = {row_bytes, rows};
  cuuint64_t strides[1] = {row_bytes};
  cuuint32_t box[2] = {128, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? LQ_OK : LQ_ERR_CUDA;
}

lq_status lq_make_tmap_rows16(CUtensorMap* tm, const void* X, uint64_t M, uint64_t K) {
  encode_tiled_fn fn = get_encode_fn();
  if (!fn) return LQ_ERR_CUDA;
  cuuint64_t dims[2] = {K, M};
  cuuint64_t strides[1] = {K * 2};
  cuuint32_t box[2] = {64, 16};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(X), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? LQ_OK : LQ_ERR_CUDA;
}

// ---- device status word ------------------------------------------------------------------
static int32_t* g_status[64] = {nullptr};
static std::mutex g_status_mu;

int32_t* lq_device_status_ptr(int device) {
  if (device < 0 || device >= 64) return nullptr;
  std::lock_guard<std::mutex> lk(g_status_mu);
  if (!g_status[device]) {
    int prev = 0;
    cudaGetDevice(&prev);
    if (cudaSetDevice(device) != cudaSuccess) return nullptr;
    int32_t* p = nullptr;
    if (cudaMalloc(&p, 2 * sizeof(int32_t)) != cudaSuccess) { cudaSetDevice(prev); return nullptr; }
    cudaMemset(p, 0, 2 * sizeof(int32_t));
    g_status[device] = p;
    cudaSetDevice(prev);
  }
  return g_status[device];
}

extern "C" lq_status lq_get_device_status(int device, int32_t* code, int32_t* stage) {
  int32_t* p = lq_device_status_ptr(device);
  if (!p) return LQ_ERR_CUDA;
  int32_t h[2] = {0, 0};
  CUDA_OK(cudaSetDevice(device));
  CUDA_OK(cudaDeviceSynchronize());
  CUDA_OK(cudaMemcpy(h, p, sizeof(h), cudaMemcpyDeviceToHost));
  CUDA_OK(cudaMemset(p, 0, sizeof(h)));
  if (code) *code = h[0];
  if (stage) *stage = h[1];
  return LQ_OK;
}

extern "C" lq_status lq_selftest_wait_timeout(int device, void* stream) {
  return lq_launch_wait_probe(device, (cudaStream_t)stream);
}

// ---- upload ------------------------------------------------------------------------------
static void layer_free_device(lq_layer* L) {
  if (L->device < 0) return;
  cudaSetDevice(L->device);
  cudaFree(L->d_Wq8); cudaFree(L->d_sw); cudaFree(L->d_L1f); cudaFree(L->d_L1h); cudaFree(L->d_sL1);
  cudaFree(L->d_L2c); cudaFree(L->d_sL2); cudaFree(L->d_bias); cudaFree(L->d_sfb);
  cudaFree(L->d_s1b); cudaFree(L->d_sfl2);
  L->d_s1b = nullptr; L->d_sfl2 = nullptr;
  L->d_Wq8 = nullptr; L->d_sw = nullptr; L->d_L1f = nullptr; L->d_L1h = nullptr; L->d_sL1 = nullptr;
  L->d_L2c = nullptr; L->d_sL2 = nullptr; L->d_bias = nullptr; L->d_sfb = nullptr;
  L->device = -1;
}

template <typename T>
static lq_status upload(T** dptr, const std::vector<T>& h) {
  if (cudaMalloc((void**)dptr, h.size() * sizeof(T)) != cudaSuccess) return LQ_ERR_ALLOC;
  CUDA_OK(cudaMemcpy(*dptr, h.data(), h.size() * sizeof(T), cudaMemcpyHostToDevice));
  return LQ_OK;
}

extern "C" lq_status lq_layer_to_device(lq_layer* L, int device) {
  if (!L) return LQ_ERR_INVALID_ARG;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return LQ_ERR_CUDA;
  layer_free_device(L);
  CUDA_OK(cudaSetDevice(device));
  L->device = device;
  L->main_kind = g_lq_main_kind;
  const int K = L->K, N = L->N, r = L->r, G = L->G, Kpad = L->Kpad, Npad = L->Npad, Gpad = L->Gpad;
  lq_status st;
  try {
    std::vector<uint8_t> w8((size_t)Npad * Kpad, lq_encode_code_host(0, L->main_kind));
    for (int k = 0; k < K; ++k)
      for (int n = 0; n < N; ++n)
        w8[(size_t)n * Kpad + k] = L->mxfp ? L->Wq8h[(size_t)k * N + n] : lq_encode_code_host(L->Wq[(size_t)k * N + n], L->main_kind);
    if ((st = upload(&L->d_Wq8, w8)) != LQ_OK) return st;
    if (L->mx) {
      // E8M0 bytes (exponent + 127) in the layout the block-scaled MMA reads from tensor memory; 127 = 2^0 for padding
      std::vector<uint8_t> sfb((size_t)(Npad / 128) * (Kpad / 128) * 512, 127);
      for (int g = 0; g < G; ++g)
        for (int n = 0; n < N; ++n) {
          int x = 0;
          frexpf(h2f(L->sw[(size_t)g * N + n]), &x);              // 2^e = 0.5 * 2^(e+1)
          sfb[lq_sfb_offset(n, g, Npad)] = (uint8_t)(x - 1 + 127);
        }
      if ((st = upload(&L->d_sfb, sfb)) != LQ_OK) return st;
    } else {
      std::vector<float> swf((size_t)Gpad * Npad, 0.f);
      for (int g = 0; g < G; ++g)
        for (int n = 0; n < N; ++n) swf[(size_t)g * Npad + n] = h2f(L->sw[(size_t)g * N + n]);
      if ((st = upload(&L->d_sw, swf)) != LQ_OK) return st;
    }
    std::vector<float> bias((size_t)Npad, 0.f);
    if (L->has_bias) for (int n = 0; n < N; ++n) bias[n] = h2f(L->bias[n]);
    if ((st = upload(&L->d_bias, bias)) != LQ_OK) return st;
    std::vector<float> s1(LQ_MAX_RANK, 1.f), s2((size_t)Npad, 1.f);
    std::vector<uint8_t> l2c((size_t)Npad * LQ_RCONT, 0);
    if (L->integer_branch) {
      // B fragments of mma.sync.m16n8k32 (s8) under the k order the quantizer's lanes hold their codes in: per box of
      // 64 values and 8-column tile, lane 4 c + t carries k = 64 box + 16 t + 0..15 of column 8 tile + c
      const int ntiles = lq_quant_rank_tiles(r, false), nbox = Kpad / 64;
      std::vector<uint8_t> l1f((size_t)nbox * ntiles * 32 * 16, 0);
      for (int b = 0; b < nbox; ++b)
        for (int nt = 0; nt < ntiles; ++nt)
          for (int lane = 0; lane < 32; ++lane) {
            const int j = nt * 8 + (lane >> 2), kb = b * 64 + (lane & 3) * 16;
            uint8_t* dst = &l1f[(((size_t)b * ntiles + nt) * 32 + lane) * 16];
            for (int i = 0; i < 16; ++i) dst[i] = (j < r && kb + i < K) ? (uint8_t)L->L1q[(size_t)(kb + i) * r + j] : 0;
          }
      if ((st = upload(&L->d_L1f, l1f)) != LQ_OK) return st;
      for (int j = 0; j < r; ++j) s1[j] = L->sL1[j];
      for (int n = 0; n < N; ++n) s2[n] = L->sL2[n];
      for (int j = 0; j < r; ++j)
        for (int n = 0; n < N; ++n) l2c[(size_t)n * LQ_RCONT + j] = (uint8_t)L->L2q[(size_t)j * N + n];
    } else if ((L->mxfp || L->a8) && r > 0) {
      // B fragments of mma.sync.m16n8k32 (e4m3) for the MXFP quantizer, whose lanes hold two runs of eight values per
      // box (one per block of 32): lane 4 c + t carries k = 64 box + 32 j + 8 t + 0..7 of column 8 tile + c, j = 0, 1
      const int ntiles = lq_quant_rank_tiles(r, false), nbox = Kpad / 64, rpad = ntiles * 8;
      std::vector<uint8_t> l1f((size_t)nbox * ntiles * 32 * 16, 0);
      for (int b = 0; b < nbox; ++b)
        for (int nt = 0; nt < ntiles; ++nt)
          for (int lane = 0; lane < 32; ++lane) {
            const int j = nt * 8 + (lane >> 2);
            uint8_t* dst = &l1f[(((size_t)b * ntiles + nt) * 32 + lane) * 16];
            for (int blk = 0; blk < 2; ++blk)
              for (int i = 0; i < 8; ++i) {
                const int k = b * 64 + 32 * blk + 8 * (lane & 3) + i;
                dst[8 * blk + i] = (j < r && k < K) ? (L->a8 ? (uint8_t)L->L1q[(size_t)k * r + j] : L->L1e[(size_t)k * r + j]) : 0;
              }
          }
      if ((st = upload(&L->d_L1f, l1f)) != LQ_OK) return st;
      std::vector<float> s1b((size_t)(Kpad / 32) * rpad, 0.f);
      for (int b = 0; b < lq_ceil_div(K, 32); ++b)
        for (int j = 0; j < r; ++j) s1b[(size_t)b * rpad + j] = L->s1b[(size_t)b * r + j];
      if ((st = upload(&L->d_s1b, s1b)) != LQ_OK) return st;
      // E8M0 bytes of L2's block scales along the rank, one 128-byte-of-rank stage: [1][Npad/128][512]
      std::vector<uint8_t> sfl2((size_t)(Npad / 128) * 512, 127);
      if (L->a8 && L->cfg.branch == LQ_BRANCH_MXINT4) {
        // 4-bit codes are their own lo digit: one plane, K blocks in order (the intermediate brings its two planes as two
        // stages against this one)
        for (int j = 0; j < r; ++j)
          for (int n = 0; n < N; ++n) l2c[(size_t)n * LQ_RCONT + j] = lq_digit_e4m3(L->L2q[(size_t)j * N + n]);
        for (int c = 0; c < lq_ceil_div(r, 32); ++c)
          for (int n = 0; n < N; ++n) {
            int e = 0;
            pow2_exponent(L->s2b[(size_t)c * N + n], &e);
            sfl2[lq_sfb_offset(n, c, Npad)] = (uint8_t)(e + 127);
          }
      } else if (L->a8) {
        // two digit planes, code = 16 hi + lo: hi digits of rank index j at byte j, lo digits at byte 64 + j (rank <= 64);
        // the four 32-byte K blocks of the stage are (hi, block 0), (hi, block 1), (lo, block 0), (lo, block 1) with
        // scales 2^(e+4), 2^(e+4), 2^e, 2^e
        for (int j = 0; j < r; ++j)
          for (int n = 0; n < N; ++n) {
            int hi, lo;
            lq_split_digits(L->L2q[(size_t)j * N + n], &hi, &lo);
            l2c[(size_t)n * LQ_RCONT + j] = lq_digit_e4m3(hi);
            l2c[(size_t)n * LQ_RCONT + 64 + j] = lq_digit_e4m3(lo);
          }
        for (int c = 0; c < lq_ceil_div(r, 32); ++c)
          for (int n = 0; n < N; ++n) {
            int e = 0;
            pow2_exponent(L->s2b[(size_t)c * N + n], &e);
            sfl2[lq_sfb_offset(n, c, Npad)] = (uint8_t)(e + 4 + 127);
            sfl2[lq_sfb_offset(n, 2 + c, Npad)] = (uint8_t)(e + 127);
          }
      } else {
        for (int j = 0; j < r; ++j)
          for (int n = 0; n < N; ++n) l2c[(size_t)n * LQ_RCONT + j] = L->L2e[(size_t)j * N + n];
        for (int c = 0; c < lq_ceil_div(r, 32); ++c)
          for (int n = 0; n < N; ++n) {
            int e = 0;
            pow2_exponent(L->s2b[(size_t)c * N + n], &e);
            sfl2[lq_sfb_offset(n, c, Npad)] = (uint8_t)(e + 127);
          }
      }
      if ((st = upload(&L->d_sfl2, sfl2)) != LQ_OK) return st;
    } else if (L->f16_branch) {
      // the same fragment order with 16 halves per lane (mma.sync.m16n8k16, four k steps per box)
      const int ntiles = lq_quant_rank_tiles(r, true), nbox = Kpad / 64;
      std::vector<uint16_t> l1t((size_t)nbox * ntiles * 32 * 16, 0);
      for (int b = 0; b < nbox; ++b)
        for (int nt = 0; nt < ntiles; ++nt)
          for (int lane = 0; lane < 32; ++lane) {
            const int j = nt * 8 + (lane >> 2), kb = b * 64 + (lane & 3) * 16;
            uint16_t* dst = &l1t[(((size_t)b * ntiles + nt) * 32 + lane) * 16];
            for (int i = 0; i < 16; ++i) dst[i] = (j < r && kb + i < K) ? L->L1h[(size_t)(kb + i) * r + j] : 0;
          }
      if ((st = upload(&L->d_L1h, l1t)) != LQ_OK) return st;
      uint16_t* c16 = (uint16_t*)l2c.data();
      for (int j = 0; j < r; ++j)
        for (int n = 0; n < N; ++n) c16[(size_t)n * (LQ_RCONT / 2) + j] = L->L2h[(size_t)j * N + n];
    }
    if ((st = upload(&L->d_sL1, s1)) != LQ_OK) return st;
    if ((st = upload(&L->d_sL2, s2)) != LQ_OK) return st;
    if ((st = upload(&L->d_L2c, l2c)) != LQ_OK) return st;
  } catch (const std::bad_alloc&) { return LQ_ERR_ALLOC; }
  if ((st = lq_make_tmap_bytes(&L->tmB, L->d_Wq8, Npad, Kpad, LQ_BN)) != LQ_OK) return st;
  if ((st = lq_make_tmap_bytes(&L->tmB2, L->d_Wq8, Npad, Kpad, 2 * LQ_BN)) != LQ_OK) return st;
  if ((st = lq_make_tmap_bytes(&L->tmL2, L->d_L2c, Npad, LQ_RCONT, LQ_BN)) != LQ_OK) return st;
  if (!lq_device_status_ptr(device)) return LQ_ERR_CUDA;
  if ((st = lq_gemm_prepare(device)) != LQ_OK) return st;
  if (L->mx && (st = lq_gemm_mx_prepare(device)) != LQ_OK) return st;
  return LQ_OK;
}

extern "C" lq_status lq_layer_free(lq_layer* L) {
  if (!L) return LQ_ERR_INVALID_ARG;
  layer_free_device(L);
  delete L;
  return LQ_OK;
}

// ---- activation record -------------------------------------------------------------------
extern "C" lq_status lq_act_create(const lq_layer* L, int32_t M_max, int device, lq_act** out) {
  if (!L || !out || M_max <= 0) return LQ_ERR_INVALID_ARG;
  if (L->device != device) return LQ_ERR_INVALID_ARG;
  lq_act* A = new (std::nothrow) lq_act();
  if (!A) return LQ_ERR_ALLOC;
  memset(A, 0, sizeof(*A));
  A->K = L->K; A->N = L->N; A->r = L->r; A->G = L->G; A->Kpad = L->Kpad; A->Gpad = L->Gpad;
  A->mx = L->mx; A->mxfp = L->mxfp; A->a8 = L->a8; A->planes = L->a8 ? 2 : 1;
  A->tq_stride = (L->a8 && L->cfg.branch == LQ_BRANCH_MXINT4) ? 2 * LQ_RCONT : LQ_RCONT;
  A->branch = L->cfg.branch; A->M_max = M_max; A->Mpad = lq_round_up(M_max, LQ_BM);
  A->device = device; A->main_kind = L->main_kind; A->M = 0;
  if (cudaSetDevice(device) != cudaSuccess) { delete A; return LQ_ERR_CUDA; }
  const size_t Mp = A->Mpad, Kp = A->Kpad, Kx = (size_t)A->planes * Kp;   // Kx: bytes per row of the main codes
  bool ok = cudaMalloc((void**)&A->d_qx8, Mp * Kx) == cudaSuccess &&
            cudaMalloc((void**)&A->d_sx, (size_t)A->Gpad * Mp * sizeof(float)) == cudaSuccess &&
            cudaMalloc((void**)&A->d_qb, Mp * Kp) == cudaSuccess &&
            cudaMalloc((void**)&A->d_sXb, Mp * sizeof(float)) == cudaSuccess &&
            cudaMalloc((void**)&A->d_tq, Mp * A->tq_stride) == cudaSuccess &&
            cudaMalloc((void**)&A->d_sT, Mp * sizeof(float)) == cudaSuccess &&
            (!A->mx || cudaMalloc((void**)&A->d_sfa, (Mp / 128) * (Kx / 128) * 512) == cudaSuccess) &&
            (!(A->mxfp || A->a8) || cudaMalloc((void**)&A->d_sft, (Mp / 128) * 512 * (A->tq_stride / LQ_RCONT)) == cudaSuccess);
  if (!ok) { lq_act_free(A); return LQ_ERR_ALLOC; }
  // padding rows/columns are read by the GEMM's tiles: start from defined contents
  cudaMemset(A->d_qx8, 0, Mp * Kx);
  cudaMemset(A->d_sx, 0, (size_t)A->Gpad * Mp * sizeof(float));
  cudaMemset(A->d_qb, 0, Mp * Kp);
  cudaMemset(A->d_sXb, 0, Mp * sizeof(float));
  cudaMemset(A->d_tq, 0, Mp * A->tq_stride);
  cudaMemset(A->d_sT, 0, Mp * sizeof(float));
  if (A->mx) cudaMemset(A->d_sfa, 127, (Mp / 128) * (Kx / 128) * 512);
  if (A->mxfp || A->a8) cudaMemset(A->d_sft, 127, (Mp / 128) * 512 * (A->tq_stride / LQ_RCONT));
  lq_status st;
  if ((st = lq_make_tmap_bytes(&A->tmA, A->d_qx8, Mp, Kx, LQ_BM)) != LQ_OK) { lq_act_free(A); return st; }
  if ((st = lq_make_tmap_bytes(&A->tmT, A->d_tq, Mp, (uint64_t)A->tq_stride, LQ_BM)) != LQ_OK) { lq_act_free(A); return st; }
  if (cudaDeviceSynchronize() != cudaSuccess) { lq_act_free(A); return LQ_ERR_CUDA; }
  *out = A;
  return LQ_OK;
}

extern "C" lq_status lq_act_free(lq_act* A) {
  if (!A) return LQ_ERR_INVALID_ARG;
  cudaSetDevice(A->device);
  cudaFree(A->d_qx8); cudaFree(A->d_sx); cudaFree(A->d_qb); cudaFree(A->d_sXb); cudaFree(A->d_tq); cudaFree(A->d_sT); cudaFree(A->d_sfa); cudaFree(A->d_sft);
  cudaFree(A->d_Xstage); cudaFree(A->d_Ystage);
  if (A->pipe_ready) {
    cudaStreamDestroy(A->s_h2d); cudaStreamDestroy(A->s_d2h);
    for (int c = 0; c < LQ_HOST_CHUNKS; ++c) { cudaEventDestroy(A->ev_x[c]); cudaEventDestroy(A->ev_y[c]); }
    cudaEventDestroy(A->ev_begin); cudaEventDestroy(A->ev_end);
  }
  delete A;
  return LQ_OK;
}

static bool act_matches(const lq_layer* L, const lq_act* A) {
  return L && A && L->device == A->device && L->device >= 0 && L->K == A->K && L->N == A->N && L->r == A->r &&
         L->cfg.branch == A->branch && L->main_kind == A->main_kind && L->mx == A->mx && L->mxfp == A->mxfp && L->a8 == A->a8;
}

extern "C" lq_status lq_quantize_act(const lq_layer* L, const void* X, int32_t M, lq_act* A, void* stream) {
  if (!L || !A || !X) return LQ_ERR_INVALID_ARG;
  if (!act_matches(L, A)) return LQ_ERR_INVALID_ARG;
  if (M <= 0 || M > A->M_max) return LQ_ERR_INVALID_ARG;
  if (((uintptr_t)X & 15) != 0) return LQ_ERR_INVALID_ARG;
  A->M = M;
  return lq_launch_quantize(L, X, M, A, (cudaStream_t)stream);
}

extern "C" lq_status lq_linear_forward(const lq_layer* L, const lq_act* A, void* Y, lq_out_dtype dt, void* stream) {
  if (!L || !A || !Y) return LQ_ERR_INVALID_ARG;
  if (!act_matches(L, A)) return LQ_ERR_INVALID_ARG;
  if (A->M <= 0) return LQ_ERR_INVALID_ARG;
  if (dt != LQ_OUT_F16 && dt != LQ_OUT_F32) return LQ_ERR_INVALID_ARG;
  if (((uintptr_t)Y & 15) != 0) return LQ_ERR_INVALID_ARG;
  return L->mx ? lq_launch_gemm_mx(L, A, Y, dt, (cudaStream_t)stream) : lq_launch_gemm(L, A, Y, dt, (cudaStream_t)stream);
}

static lq_status forward_host(const lq_layer* L, lq_act* A, const void* Xh, int32_t M, void* Yh, lq_out_dtype dt, void* stream,
                              bool wait) {
  if (!L || !A || !Xh || !Yh) return LQ_ERR_INVALID_ARG;
  if (!act_matches(L, A)) return LQ_ERR_INVALID_ARG;
  if (M <= 0 || M > A->M_max) return LQ_ERR_INVALID_ARG;
  if (dt != LQ_OUT_F16 && dt != LQ_OUT_F32) return LQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  CUDA_OK(cudaSetDevice(A->device));
  if (!A->d_Xstage && cudaMalloc(&A->d_Xstage, (size_t)A->M_max * A->K * 2) != cudaSuccess) return LQ_ERR_ALLOC;
  // sized once, for the wider output type: it is never freed or re-allocated while an earlier call's copies
  // may still be queued
  const size_t ybytes = (size_t)A->M_max * A->N * 4;
  if (!A->d_Ystage) {
    if (cudaMalloc(&A->d_Ystage, ybytes) != cudaSuccess) return LQ_ERR_ALLOC;
    A->ystage_bytes = ybytes;
  }
  // Rows are independent, so the call is pipelined over row chunks: while chunk c is computed on the caller's
  // stream, chunk c+1 travels host -> device and chunk c-1 device -> host on two copy streams.
  if (!A->pipe_ready) {
    CUDA_OK(cudaStreamCreateWithFlags(&A->s_h2d, cudaStreamNonBlocking));
    CUDA_OK(cudaStreamCreateWithFlags(&A->s_d2h, cudaStreamNonBlocking));
    for (int c = 0; c < LQ_HOST_CHUNKS; ++c) {
      CUDA_OK(cudaEventCreateWithFlags(&A->ev_x[c], cudaEventDisableTiming));
      CUDA_OK(cudaEventCreateWithFlags(&A->ev_y[c], cudaEventDisableTiming));
    }
    CUDA_OK(cudaEventCreateWithFlags(&A->ev_begin, cudaEventDisableTiming));
    CUDA_OK(cudaEventCreateWithFlags(&A->ev_end, cudaEventDisableTiming));
    A->pipe_ready = true;
  }
  const int nchunk = std::max(1, std::min(LQ_HOST_CHUNKS, M / (2 * LQ_BM)));   // chunks of at least 256 rows
  const int rows_per = lq_round_up(lq_ceil_div(M, nchunk), LQ_BM);
  const size_t esz = dt == LQ_OUT_F32 ? 4 : 2;
  CUDA_OK(cudaEventRecord(A->ev_begin, st));                  // copies start after what the caller queued before
  CUDA_OK(cudaStreamWaitEvent(A->s_h2d, A->ev_begin, 0));
  CUDA_OK(cudaStreamWaitEvent(A->s_d2h, A->ev_begin, 0));
  for (int c = 0; c < nchunk; ++c) {
    const int m0 = c * rows_per;
    if (m0 >= M) break;
    const int Mc = M - m0 < rows_per ? M - m0 : rows_per;
    const uint8_t* xh = (const uint8_t*)Xh + (size_t)m0 * A->K * 2;
    uint8_t* xd = (uint8_t*)A->d_Xstage + (size_t)m0 * A->K * 2;
    uint8_t* yd = (uint8_t*)A->d_Ystage + (size_t)m0 * A->N * esz;
    CUDA_OK(cudaMemcpyAsync(xd, xh, (size_t)Mc * A->K * 2, cudaMemcpyHostToDevice, A->s_h2d));
    CUDA_OK(cudaEventRecord(A->ev_x[c], A->s_h2d));
    CUDA_OK(cudaStreamWaitEvent(st, A->ev_x[c], 0));
    // a view of the activation record that starts at row m0 (m0 is a multiple of the row tile)
    lq_act V = *A;
    V.M = Mc; V.M_max = Mc;
    V.d_qx8 = A->d_qx8 + (size_t)m0 * A->Kpad * A->planes;
    V.d_qb = A->d_qb + (size_t)m0 * A->Kpad;
    V.d_sx = A->d_sx + m0;                                     // [Gpad][Mpad]: the row stride stays Mpad
    V.d_sXb = A->d_sXb + m0;
    V.d_tq = A->d_tq + (size_t)m0 * A->tq_stride;
    V.d_sT = A->d_sT + m0;
    if (A->mx) V.d_sfa = A->d_sfa + (size_t)(m0 / 128) * (A->Kpad / 128) * A->planes * 512;
    if (A->mxfp || A->a8) V.d_sft = A->d_sft + (size_t)(m0 / 128) * 512 * (A->tq_stride / LQ_RCONT);
    lq_status s;
    if ((s = lq_make_tmap_bytes(&V.tmA, V.d_qx8, (uint64_t)(A->Mpad - m0), (uint64_t)A->Kpad * A->planes, LQ_BM)) != LQ_OK) return s;
    if ((s = lq_make_tmap_bytes(&V.tmT, V.d_tq, (uint64_t)(A->Mpad - m0), (uint64_t)A->tq_stride, LQ_BM)) != LQ_OK) return s;
    if ((s = lq_launch_quantize(L, xd, Mc, &V, st)) != LQ_OK) return s;
    if ((s = (L->mx ? lq_launch_gemm_mx(L, &V, yd, dt, st) : lq_launch_gemm(L, &V, yd, dt, st))) != LQ_OK) return s;
    CUDA_OK(cudaEventRecord(A->ev_y[c], st));
    CUDA_OK(cudaStreamWaitEvent(A->s_d2h, A->ev_y[c], 0));
    CUDA_OK(cudaMemcpyAsync((uint8_t*)Yh + (size_t)m0 * A->N * esz, yd, (size_t)Mc * A->N * esz, cudaMemcpyDeviceToHost, A->s_d2h));
  }
  A->M = M;
  CUDA_OK(cudaEventRecord(A->ev_end, A->s_d2h));
  CUDA_OK(cudaStreamWaitEvent(st, A->ev_end, 0));              // the caller's stream is done when Y has arrived
  if (wait) CUDA_OK(cudaStreamSynchronize(st));
  return LQ_OK;
}

extern "C" lq_status lq_linear_forward_host(const lq_layer* L, lq_act* A, const void* Xh, int32_t M, void* Yh,
                                            lq_out_dtype dt, void* stream) {
  return forward_host(L, A, Xh, M, Yh, dt, stream, true);
}

extern "C" lq_status lq_linear_forward_host_async(const lq_layer* L, lq_act* A, const void* Xh, int32_t M, void* Yh,
                                                  lq_out_dtype dt, void* stream) {
  return forward_host(L, A, Xh, M, Yh, dt, stream, false);
}

static int decode_code(uint8_t b, int kind) {
  if (kind == LQ_KIND_I8) return (int)(int8_t)b;
  int mag = 0;
  switch (b & 0x7F) {
    case 0x00: mag = 0; break; case 0x38: mag = 1; break; case 0x40: mag = 2; break; case 0x44: mag = 3; break;
    case 0x48: mag = 4; break; case 0x4A: mag = 5; break; case 0x4C: mag = 6; break; case 0x4E: mag = 7; break;
    default: mag = 99; break;   // not a code byte: surfaces as a parity failure
  }
  return (b & 0x80) ? -mag : mag;
}

// value of a digit byte written by the MXINT8 quantizer (an E4M3 image of an integer in [-8, 8])
static int decode_digit(uint8_t b) {
  for (int d = -8; d <= 8; ++d)
    if (lq_digit_e4m3(d) == b) return d;
  return (b & 0x7F) == 0 ? 0 : 99;   // -0 reads as 0; anything else surfaces as a parity failure
}

extern "C" lq_status lq_act_export(const lq_act* A, int8_t* qx, uint16_t* sx, int8_t* qb, float* sXb, void* tq,
                                   float* sT, void* stream) {
  if (!A || A->M <= 0) return LQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  CUDA_OK(cudaSetDevice(A->device));
  CUDA_OK(cudaStreamSynchronize(st));
  const int M = A->M, K = A->K, G = A->G, r = A->r;
  const size_t Kp = A->Kpad, Mp = A->Mpad;
  try {
    if (qx && A->a8) {
      std::vector<uint8_t> h((size_t)M * 2 * Kp);
      CUDA_OK(cudaMemcpy(h.data(), A->d_qx8, h.size(), cudaMemcpyDeviceToHost));
      for (int m = 0; m < M; ++m)
        for (int k = 0; k < K; ++k)
          qx[(size_t)m * K + k] = (int8_t)(16 * decode_digit(h[(size_t)m * 2 * Kp + k]) + decode_digit(h[(size_t)m * 2 * Kp + Kp + k]));
    } else if (qx) {
      std::vector<uint8_t> h((size_t)M * Kp);
      CUDA_OK(cudaMemcpy(h.data(), A->d_qx8, h.size(), cudaMemcpyDeviceToHost));
      for (int m = 0; m < M; ++m)
        for (int k = 0; k < K; ++k)   // MXFP: the e4m3 bytes themselves
          qx[(size_t)m * K + k] = A->mxfp ? (int8_t)h[m * Kp + k] : (int8_t)decode_code(h[m * Kp + k], A->main_kind);
    }
    if (sx && A->mx) {
      const size_t Kx = (size_t)A->planes * Kp;                   // a8: the lo plane's scale bytes carry e itself
      std::vector<uint8_t> h((Mp / 128) * (Kx / 128) * 512);
      CUDA_OK(cudaMemcpy(h.data(), A->d_sfa, h.size(), cudaMemcpyDeviceToHost));
      for (int m = 0; m < M; ++m)
        for (int g = 0; g < G; ++g) {
          const int e = (int)h[lq_sf_offset(m, g + (A->a8 ? (int)(Kp / 32) : 0), (int)Kx)] - 127;
          sx[(size_t)m * G + g] = (uint16_t)(int16_t)e;            // MXINT4: the block exponent itself (scale 2^e)
        }
    } else if (sx) {
      std::vector<float> h((size_t)A->Gpad * Mp);
      CUDA_OK(cudaMemcpy(h.data(), A->d_sx, h.size() * sizeof(float), cudaMemcpyDeviceToHost));
      for (int m = 0; m < M; ++m)
        for (int g = 0; g < G; ++g) {
          __half v = __float2half_rn(h[(size_t)g * Mp + m]);   // exact: the value is an fp16 number
          sx[(size_t)m * G + g] = __half_raw(v).x;
        }
    }
    if (qb && A->branch != LQ_BRANCH_NONE && A->branch != LQ_BRANCH_W16A16 && !A->mxfp && !A->a8) {
      std::vector<int8_t> h((size_t)M * Kp);
      CUDA_OK(cudaMemcpy(h.data(), A->d_qb, h.size(), cudaMemcpyDeviceToHost));
      for (int m = 0; m < M; ++m) memcpy(qb + (size_t)m * K, h.data() + m * Kp, K);
    }
    if (sXb && r > 0 && !A->mxfp && !A->a8) CUDA_OK(cudaMemcpy(sXb, A->d_sXb, M * sizeof(float), cudaMemcpyDeviceToHost));
    if (tq && r > 0) {
      const size_t ts = (size_t)A->tq_stride, lo_at = ts / 2;     // a8: the lo digits sit half a container row after the hi digits
      std::vector<uint8_t> h((size_t)M * ts);
      CUDA_OK(cudaMemcpy(h.data(), A->d_tq, h.size(), cudaMemcpyDeviceToHost));
      const int eb = A->branch == LQ_BRANCH_W16A16 ? 2 : 1;
      if (A->a8) {
        for (int m = 0; m < M; ++m)
          for (int j = 0; j < r; ++j)
            ((int8_t*)tq)[(size_t)m * r + j] =
                (int8_t)(16 * decode_digit(h[(size_t)m * ts + j]) + decode_digit(h[(size_t)m * ts + lo_at + j]));
      } else {
        for (int m = 0; m < M; ++m) memcpy((uint8_t*)tq + (size_t)m * r * eb, h.data() + (size_t)m * ts, (size_t)r * eb);
      }
    }
    if (sT && r > 0 && A->a8) {
      // the block exponents of the rank-r intermediate (the lo plane's scale bytes), as floats [M][ceil(r/32)]
      const bool split = A->tq_stride != LQ_RCONT;                // two chunks per row block: hi plane, lo plane
      std::vector<uint8_t> h((Mp / 128) * 512 * (split ? 2 : 1));
      CUDA_OK(cudaMemcpy(h.data(), A->d_sft, h.size(), cudaMemcpyDeviceToHost));
      const int nbR = lq_ceil_div(r, LQ_MX_BLOCK);
      for (int m = 0; m < M; ++m)
        for (int c = 0; c < nbR; ++c)
          sT[(size_t)m * nbR + c] = (float)((int)h[split ? lq_sf_offset(m, 4 + c, 256) : lq_sf_offset(m, 2 + c, 128)] - 127);
    } else if (sT && r > 0 && A->mxfp) {
      // MXFP: the block exponents of the rank-r intermediate as floats, [M][ceil(r/32)]
      std::vector<uint8_t> h((Mp / 128) * 512);
      CUDA_OK(cudaMemcpy(h.data(), A->d_sft, h.size(), cudaMemcpyDeviceToHost));
      const int nbR = lq_ceil_div(r, LQ_MX_BLOCK);
      for (int m = 0; m < M; ++m)
        for (int c = 0; c < nbR; ++c) sT[(size_t)m * nbR + c] = (float)((int)h[lq_sf_offset(m, c, 128)] - 127);
    } else if (sT && r > 0) CUDA_OK(cudaMemcpy(sT, A->d_sT, M * sizeof(float), cudaMemcpyDeviceToHost));
  } catch (const std::bad_alloc&) { return LQ_ERR_ALLOC; }
  return LQ_OK;
}
