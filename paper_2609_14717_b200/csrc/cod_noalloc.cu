// cod_lm_head_argmax_static: the LM-head argmax without a context and without any allocation.
//
// Who needs this: callers that are not allowed to call cudaMalloc (or cod_create, which does).
// Typical cases are a serving process that has handed all device memory to its own pool and must
// not let a library carve out more behind its back, and a latency-critical decode loop in which
// cudaMalloc's device-wide synchronisation would stall every other stream. For them the scratch
// this operation needs (the normalised activations and the packed per-row argmax keys) lives in a
// fixed array that is part of the library image: every GPU that loads the library holds
// COD_STATIC_SCRATCH_BYTES of it until the process exits.
//
// Consequences the caller must know:
//   * sizes are capped (COD_STATIC_MAX_ROWS rows, COD_STATIC_MAX_DMODEL columns); larger requests
//     are refused with COD_ERR_TOO_LARGE, nothing is launched;
//   * all calls on one device share the one array, and it keeps the previous call's contents. The
//     kernels clear what has to start at zero (the argmax keys) themselves, but two calls whose
//     kernels overlap on the GPU (different streams, no dependency) race on the scratch;
//   * the first call on each device looks up the array's device address (cudaGetSymbolAddress,
//     with that device current). Make that first call before any stream capture begins;
//   * there is no context, hence no status word to poll: a row whose contraction did not complete
//     (a bounded device wait that ran out) comes back as tok = -1, every other row as a token id in
//     [0, vocab). Callers that need to know check for negative tokens.
#include <string.h>

#include "cod_internal.cuh"

#define COD_STATIC_MAX_ROWS 64
#define COD_STATIC_MAX_DMODEL 8192
#define COD_STATIC_ACT_BYTES (COD_STATIC_MAX_ROWS * COD_STATIC_MAX_DMODEL * 4)   /* activations, up to float */
#define COD_STATIC_KEY_BYTES (COD_STATIC_MAX_ROWS * 8)                           /* packed argmax keys        */
#define COD_STATIC_SCRATCH_BYTES (COD_STATIC_ACT_BYTES + COD_STATIC_KEY_BYTES + 256)

namespace {

// In host code this name is only a handle for the symbol, not a device address: a kernel must be
// given the pointer that cudaGetSymbolAddress returns for the current device.
static __device__ __align__(256) unsigned char g_static_scratch[COD_STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
unsigned char* g_scratch_addr[MAX_DEVICES];   // per device, filled on first use
int g_sm_count[MAX_DEVICES];                  // per device, filled with the address

int scratch_for_current_device(unsigned char** out, int* n_sm) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return COD_ERR_CUDA;
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    int sms = 0;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
      cudaGetLastError();
      return COD_ERR_CUDA;
    }
    g_sm_count[dev] = sms;
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_addr[dev];
  *n_sm = g_sm_count[dev];
  return COD_OK;
}

}  // namespace

extern "C" int cod_lm_head_argmax_static(const void* emb, const void* g_final, const float* x, int n_rows,
                                         int d_model, int vocab, int dtype, float rms_eps, int32_t* tok,
                                         float* top_logit, cod_stream_t stream) {
  if (!emb || !g_final || !x || !tok) return COD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(emb) | reinterpret_cast<uintptr_t>(g_final) | reinterpret_cast<uintptr_t>(x)) & 15u)
    return COD_ERR_INVALID_ARG;
  if (dtype != COD_F32 && dtype != COD_BF16) return COD_ERR_INVALID_ARG;
  if (n_rows < 1 || d_model < 8 || d_model % 8 || vocab < 2 || !(rms_eps >= 0.f)) return COD_ERR_INVALID_ARG;
  if (n_rows > COD_STATIC_MAX_ROWS || d_model > COD_STATIC_MAX_DMODEL) return COD_ERR_TOO_LARGE;

  unsigned char* scratch = nullptr;
  int n_sm = 0;
  int rc = scratch_for_current_device(&scratch, &n_sm);
  if (rc != COD_OK) return rc;

  // A context on the stack that points the existing kernels at the static scratch. Nothing here
  // allocates: the launchers below only read these fields.
  cod_ctx c;
  memset(&c, 0, sizeof(c));
  c.cfg.d_model = d_model;
  c.cfg.vocab = vocab;
  c.cfg.dtype = dtype;
  c.cfg.rms_eps = rms_eps;
  c.cfg.block = 1;
  c.D = d_model;
  c.R_max = COD_STATIC_MAX_ROWS;
  c.n_sm = n_sm;
  c.w.emb = emb;
  c.w.g_final = g_final;
  c.has_weights = true;
  c.a = scratch;
  c.amax = reinterpret_cast<unsigned long long*>(scratch + COD_STATIC_ACT_BYTES);
  c.status = reinterpret_cast<uint32_t*>(scratch + COD_STATIC_ACT_BYTES + COD_STATIC_KEY_BYTES);
  if (cudaGetDevice(&c.device) != cudaSuccess) return COD_ERR_CUDA;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // N_f(x) into the scratch; this kernel also resets the argmax keys of the rows it handles
  if ((rc = cod_launch_resid_norm(&c, nullptr, 0, n_rows, const_cast<float*>(x), g_final, nullptr, st)) != COD_OK) return rc;
  GemmArgs g{};
  g.A = c.a; g.lda = d_model; g.n_rows = n_rows; g.K = d_model;
  g.seg[0] = {emb, vocab}; g.n_seg = 1;
  g.splits = 1; g.amax = c.amax; g.klass = COD_K_LMHEAD;
  if ((rc = cod_launch_gemm(&c, g, st)) != COD_OK) return rc;
  return cod_launch_finalize(&c, n_rows, 1, nullptr, tok, nullptr, top_logit, st);
}
