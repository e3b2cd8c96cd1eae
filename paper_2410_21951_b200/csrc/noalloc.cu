// vadusa_draft_topk_static: the draft heads' top-k with all scratch in a fixed device array.
//
// For callers that must not allocate device memory: code that runs inside another
// framework's memory plan, a real-time audio loop that may not touch the allocator after
// start-up, or a process whose device memory was handed out completely before this library
// was loaded.  The regular path (vadusa_draft) keeps the draft heads' intermediate results in
// the caller's workspace; here they live in g_static_scratch below, a file-scope device array
// of kStaticScratchBytes that every GPU which loads this library holds until the process exits.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "../../include/vadusa.h"

namespace {
// This file's own copies of the product and selection kernels (the library's main translation
// unit compiles the same headers): inside the unnamed namespace they do not clash at link time.
#include "gemm_simt.cuh"
#include "select.cuh"
using namespace vadusa;

constexpr long long kStaticScratchBytes = 2ll << 20;          // 2 MiB per GPU
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code the name g_static_scratch is only a handle for the runtime, not an address a
// kernel can use: the device address is looked up once per device and kept here.
constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {nullptr};
char g_last_error[256] = "";

vadusa_status fail(vadusa_status s, const char* msg) {
  snprintf(g_last_error, sizeof(g_last_error), "%s", msg);
  return s;
}

long long align256(long long v) { return (v + 255) / 256 * 256; }

// "sequence b is active" words for the select kernel, kept in the last 256 bytes of the array
__global__ void set_active_words(int32_t* p, int n) {
  if ((int)threadIdx.x < n) p[threadIdx.x] = 1;
}

template <typename T>
vadusa_status run(unsigned char* scratch, const void* dw, const float* db, const void* du, const void* hstar,
                  int batch, int d, int vocab, int ld, int heads, int topk, int eos_masked, int32_t* topk_out,
                  cudaStream_t stream) {
  // scratch layout: z [heads][batch][d] of T, then logits [heads][batch][ld] fp32, and the
  // active words at the very end.  All of it is fully overwritten before it is read, so
  // nothing has to be cleared between calls.
  T* z = reinterpret_cast<T*>(scratch);
  float* logits = reinterpret_cast<float*>(scratch + align256((long long)heads * batch * d * sizeof(T)));
  int32_t* active = reinterpret_cast<int32_t*>(scratch + kStaticScratchBytes - 256);
  set_active_words<<<1, 64, 0, stream>>>(active, batch);
  EpiDraftHiddenFlat<T> eh{db, reinterpret_cast<const T*>(hstar), z, d, batch};
  dim3 g1((heads * d + 63) / 64, (batch + 63) / 64, 1);
  gemm_simt_kernel<T, EpiDraftHiddenFlat<T>><<<g1, 256, 0, stream>>>(
      reinterpret_cast<const T*>(hstar), reinterpret_cast<const T*>(dw), batch, heads * d, d, 0, 0, eh);
  EpiLogits el{logits, ld, (long long)batch * ld};
  dim3 g2((ld + 63) / 64, (batch + 63) / 64, heads);
  gemm_simt_kernel<T, EpiLogits><<<g2, 256, 0, stream>>>(z, reinterpret_cast<const T*>(du), batch, ld, d,
                                                         (long long)batch * d, (long long)ld * d, el);
  SamplingDev sp = {};
  sp.tau = 1; sp.temperature = 0.f; sp.inv_temperature = 1.f; sp.top_p = 1.f;
  sp.eos_masked = eos_masked ? 1 : 0; sp.eos_id = vocab - 1;
  // grid.x = heads only: the select kernel's extra block (the root sample) is not launched
  dim3 g3(heads, batch);
  draft_select_kernel<<<g3, 256, 0, stream>>>(logits, nullptr, ld, vocab, batch, heads, topk, nullptr, active, sp,
                                              topk_out, nullptr);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(VADUSA_ECUDA, cudaGetErrorString(e));
  return VADUSA_OK;
}

}  // namespace

extern "C" {

int64_t vadusa_static_scratch_bytes(void) { return kStaticScratchBytes; }

const char* vadusa_static_last_error(void) { return g_last_error; }

vadusa_status vadusa_draft_topk_static(const void* draft_w, const float* draft_b, const void* draft_u,
                                       const void* hstar, int32_t dtype, int32_t batch, int32_t d_model,
                                       int32_t vocab, int32_t n_draft_heads, int32_t topk, int32_t eos_masked,
                                       int32_t* topk_out, void* stream) {
  if (!draft_w || !draft_b || !draft_u || !hstar || !topk_out) return fail(VADUSA_EINVAL, "a pointer argument is NULL");
  if (dtype != 0 && dtype != 1) return fail(VADUSA_EINVAL, "dtype must be 0 (fp32) or 1 (bf16)");
  if (batch < 1 || batch > 64 || d_model < 16 || d_model % 16 || vocab < 2 || n_draft_heads < 1 ||
      n_draft_heads > VADUSA_MAX_DEPTH || topk < 1 || topk > VADUSA_MAX_DRAFT_TOPK || topk >= vocab)
    return fail(VADUSA_EINVAL, "a size argument is out of range");
  const int ld = (vocab + 127) / 128 * 128;
  const long long es = dtype == 1 ? 2 : 4;
  const long long need = align256((long long)n_draft_heads * batch * d_model * es) +
                         align256((long long)n_draft_heads * batch * ld * 4) + 256;
  if (need > kStaticScratchBytes) {
    snprintf(g_last_error, sizeof(g_last_error),
             "vadusa_draft_topk_static needs %lld bytes of scratch for these sizes; the built-in array has %lld",
             need, kStaticScratchBytes);
    return VADUSA_ENOMEM;
  }
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return fail(VADUSA_ECUDA, "no current CUDA device");
  }
  if (!g_scratch_ptr[dev]) {
    // first call on this device (it is the current one): ask the runtime for the array's device address
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) { cudaGetLastError(); return fail(VADUSA_ECUDA, cudaGetErrorString(e)); }
    g_scratch_ptr[dev] = p;
  }
  unsigned char* scratch = reinterpret_cast<unsigned char*>(g_scratch_ptr[dev]);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (dtype == 1)
    return run<bf16>(scratch, draft_w, draft_b, draft_u, hstar, batch, d_model, vocab, ld, n_draft_heads, topk,
                     eos_masked, topk_out, st);
  return run<float>(scratch, draft_w, draft_b, draft_u, hstar, batch, d_model, vocab, ld, n_draft_heads, topk,
                    eos_masked, topk_out, st);
}

}  // extern "C"
