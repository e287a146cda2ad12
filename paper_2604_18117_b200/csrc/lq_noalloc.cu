// lq_linear_forward_static: the whole forward (activation quantizer, down-projection, GEMM)
// for callers that must not allocate device memory at call time.
//
// Who these callers are: an inference server that hands all device memory to its own pool
// at start-up and forbids raw allocations afterwards (a late cudaMalloc can fail or fragment
// the pool, and it synchronises the whole device, stalling every other stream); a real-time
// loop with a fixed memory budget; a plugin running inside a host framework that owns the
// allocator.  The regular path needs an lq_act record, which lq_act_create allocates.  Here the
// record lives in a fixed array that is part of the library image instead, so the call takes
// only the caller's X and Y.
//
// The array is a file-scope __device__ array: every GPU that loads the library holds its
// LQ_STATIC_SCRATCH_BYTES until the process exits.  In host code the array's name is only a
// host-side handle, not a device address, so the address is fetched with cudaGetSymbolAddress,
// once per device with that device current, on the first call for that device.
#include <string.h>

#include <mutex>

#include "lq_internal.h"

static __device__ __align__(256) unsigned char g_lq_static_scratch[LQ_STATIC_SCRATCH_BYTES];

namespace {

std::mutex g_mu;
unsigned char* g_scratch_dev[64] = {nullptr};   // device address of the array, per device

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace

extern "C" lq_status lq_linear_forward_static(const lq_layer* L, const void* X, int32_t M, void* Y, lq_out_dtype dt,
                                              void* stream) {
  if (!L || !X || !Y) return LQ_ERR_INVALID_ARG;
  if (L->device < 0 || L->device >= 64) return LQ_ERR_INVALID_ARG;      // layer not uploaded
  if (M <= 0) return LQ_ERR_INVALID_ARG;
  if (L->mx || L->mxfp) return LQ_ERR_UNSUPPORTED;                      // SINT4 layers only
  if (dt != LQ_OUT_F16 && dt != LQ_OUT_F32) return LQ_ERR_INVALID_ARG;
  if ((((uintptr_t)X) & 15) != 0 || (((uintptr_t)Y) & 15) != 0) return LQ_ERR_INVALID_ARG;

  // carve the activation record out of the fixed array
  const size_t Mpad = (size_t)lq_round_up(M, LQ_BM), Kpad = (size_t)L->Kpad, Gpad = (size_t)L->Gpad;
  size_t off = 0;
  const size_t o_qx = off; off = align256(off + Mpad * Kpad);
  const size_t o_qb = off; off = align256(off + Mpad * Kpad);
  const size_t o_sx = off; off = align256(off + Gpad * Mpad * sizeof(float));
  const size_t o_sXb = off; off = align256(off + Mpad * sizeof(float));
  const size_t o_tq = off; off = align256(off + Mpad * LQ_RCONT);
  const size_t o_sT = off; off = align256(off + Mpad * sizeof(float));
  if (off > (size_t)LQ_STATIC_SCRATCH_BYTES) return LQ_ERR_UNSUPPORTED;  // M x K too large for the fixed array

  if (lq_note_cuda(cudaSetDevice(L->device)) != cudaSuccess) return LQ_ERR_CUDA;
  unsigned char* base = nullptr;
  {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_scratch_dev[L->device]) {
      void* p = nullptr;
      if (lq_note_cuda(cudaGetSymbolAddress(&p, g_lq_static_scratch)) != cudaSuccess || !p) return LQ_ERR_CUDA;
      g_scratch_dev[L->device] = (unsigned char*)p;
    }
    base = g_scratch_dev[L->device];
  }
  cudaStream_t st = (cudaStream_t)stream;
  // The array keeps the previous call's contents; padding columns, padding rows and the tail
  // of the rank-r containers must read as zero codes, so clear the part this call uses.
  if (lq_note_cuda(cudaMemsetAsync(base, 0, off, st)) != cudaSuccess) return LQ_ERR_CUDA;

  lq_act A;
  memset(&A, 0, sizeof(A));
  A.K = L->K; A.N = L->N; A.r = L->r; A.G = L->G; A.Kpad = L->Kpad; A.Gpad = L->Gpad;
  A.branch = L->cfg.branch; A.M_max = M; A.Mpad = (int)Mpad; A.device = L->device; A.main_kind = L->main_kind; A.M = M;
  A.d_qx8 = base + o_qx;
  A.d_qb = (int8_t*)(base + o_qb);
  A.d_sx = (float*)(base + o_sx);
  A.d_sXb = (float*)(base + o_sXb);
  A.d_tq = base + o_tq;
  A.d_sT = (float*)(base + o_sT);
  lq_status s;
  if ((s = lq_make_tmap_bytes(&A.tmA, A.d_qx8, Mpad, Kpad, LQ_BM)) != LQ_OK) return s;
  if ((s = lq_make_tmap_bytes(&A.tmT, A.d_tq, Mpad, LQ_RCONT, LQ_BM)) != LQ_OK) return s;
  if ((s = lq_launch_quantize(L, X, M, &A, st)) != LQ_OK) return s;
  return lq_launch_gemm(L, &A, Y, dt, st);
}
