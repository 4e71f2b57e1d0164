// sol_attn_thresholds_static: the threshold step (pooled-key moments -> mu, sigma, tau per query
// block) for callers that cannot allocate device memory.
//
// Some hosts of this library never get to call cudaMalloc: a plugin that runs inside another
// framework's memory pool and is handed only its input and output tensors, a process whose
// device memory is fully reserved up front, or code running where an allocation would
// synchronise the device and stall a latency-critical loop.  The regular entry points keep
// their intermediate moments in a caller-provided workspace; this one keeps them in a fixed
// array that lives inside the library image on every GPU that loads it.
#include <cmath>
#include <mutex>

#include "common.cuh"

namespace {

// 4 MiB of device memory per GPU.  The array belongs to this file's CUDA module, which the runtime
// loads on a device the first time something of the module is used there: the first call of the entry
// point on a device therefore loads the module and reserves the 4 MiB (it can fail, or synchronise, like
// any module load); from then on the memory is held until the process exits and later calls touch no
// allocator.  Layout for one call: m_K [BH][d] followed by C_K [BH][d][d].
constexpr size_t kScratchFloats = size_t(1) << 20;
static __device__ __align__(256) float g_scratch[kScratchFloats];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
float* g_scratch_ptr[kMaxDevices] = {nullptr};   // device address of g_scratch, per device

// `g_scratch` in HOST code is only a handle for the runtime, not a device address; the address a
// kernel may dereference has to be asked for, once per device, with that device current.  The
// address is cached for the life of the process: a cudaDeviceReset() in between invalidates it, and
// the library must then be reloaded.
sol_status_t scratch_for_current_device(float** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SOL_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return SOL_ERR_UNSUPPORTED_SHAPE;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    float* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_scratch) != cudaSuccess || !p) {
      cudaGetLastError();                            // leave no sticky-looking error behind
      return SOL_ERR_STATIC_SCRATCH;
    }
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return SOL_OK;
}

// m_K[c] = mean_j KC[j][c].  One CTA per (batch, head), one thread per channel.
__global__ void static_key_mean(const float* __restrict__ kc, float* __restrict__ mk, int Nk, int d) {
  const int bh = blockIdx.x, c = threadIdx.x;
  const float* src = kc + (size_t)bh * Nk * d;
  float s0 = 0.f, s1 = 0.f;
  int j = 0;
  for (; j + 1 < Nk; j += 2) {
    s0 += src[(size_t)j * d + c];
    s1 += src[(size_t)(j + 1) * d + c];
  }
  if (j < Nk) s0 += src[(size_t)j * d + c];
  mk[(size_t)bh * d + c] = (s0 + s1) / (float)Nk;
}

// C_K[r][c] = mean_j (KC[j][r] - m_K[r]) (KC[j][c] - m_K[c]).  Grid (d/16, BH), 256 threads:
// thread (r, cg) owns d/16 consecutive columns of one row.  Every entry is written exactly once
// (no accumulation across CTAs), so nothing in the scratch array has to start at zero.
__global__ void __launch_bounds__(256) static_key_cov(const float* __restrict__ kc, const float* __restrict__ mk,
                                                      float* __restrict__ cov, int Nk, int d) {
  __shared__ float xs[16][128];
  const int bh = blockIdx.y;
  const int cpt = d / 16;
  const int r = blockIdx.x * 16 + threadIdx.x / 16;
  const int c0 = (threadIdx.x % 16) * cpt;
  const float* src = kc + (size_t)bh * Nk * d;
  const float* mean = mk + (size_t)bh * d;
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int j0 = 0; j0 < Nk; j0 += 16) {
    const int nj = min(16, Nk - j0);
    for (int e = threadIdx.x; e < nj * d; e += 256) {
      const int jj = e / d, c = e % d;
      xs[jj][c] = src[(size_t)(j0 + jj) * d + c] - mean[c];
    }
    __syncthreads();
    for (int jj = 0; jj < nj; ++jj) {
      const float xr = xs[jj][r];
      for (int c = 0; c < cpt; ++c) acc[c] = fmaf(xr, xs[jj][c0 + c], acc[c]);
    }
    __syncthreads();
  }
  float* dst = cov + ((size_t)bh * d + r) * d + c0;
  for (int c = 0; c < cpt; ++c) dst[c] = acc[c] / (float)Nk;
}

// mu_i = s Qbar_i . m_K, sigma_i = s sqrt(Qbar_i C_K Qbar_i^T), tau_i = mu_i + beta sigma_i.
// One warp per query block; lane l owns rows l, l+32, ... of C_K (the lanes of a warp read C_K a row
// apart, i.e. uncoalesced; the matrix is 64 KB per head and stays in cache, and this kernel is a
// fraction of a percent of a call).
__global__ void __launch_bounds__(256) static_tau(const float* __restrict__ qbar, const float* __restrict__ mk,
                                                  const float* __restrict__ cov, float* __restrict__ mu,
                                                  float* __restrict__ sigma, float* __restrict__ tau, int Nq, int d,
                                                  float scale, float beta) {
  const int bh = blockIdx.y;
  const int i = blockIdx.x * 8 + threadIdx.x / 32, lane = threadIdx.x % 32;
  if (i >= Nq) return;
  const float* q = qbar + ((size_t)bh * Nq + i) * d;
  const float* c_k = cov + (size_t)bh * d * d;
  const float* m_k = mk + (size_t)bh * d;
  float quad = 0.f, dotm = 0.f;
  for (int r = lane; r < d; r += 32) {
    float y = 0.f;
    for (int c = 0; c < d; ++c) y = fmaf(c_k[(size_t)r * d + c], q[c], y);
    quad = fmaf(q[r], y, quad);
    dotm = fmaf(q[r], m_k[r], dotm);
  }
  for (int o = 16; o > 0; o >>= 1) {
    quad += __shfl_xor_sync(0xffffffffu, quad, o);
    dotm += __shfl_xor_sync(0xffffffffu, dotm, o);
  }
  if (lane == 0) {
    const float m = scale * dotm;
    const float s = scale * sqrtf(fmaxf(quad, 0.f));
    const size_t o = (size_t)bh * Nq + i;
    mu[o] = m;
    sigma[o] = s;
    tau[o] = isinf(beta) ? beta : fmaf(beta, s, m);
  }
}

}  // namespace

extern "C" sol_status_t sol_attn_thresholds_static(const float* qbar, const float* kc, int B, int H, int Nq, int Nk,
                                                   int d, float scale, float threshold, float* mu, float* sigma,
                                                   float* tau, sol_stream_t stream) {
  if (!qbar || !kc || !mu || !sigma || !tau) return SOL_ERR_INVALID_ARG;
  if (B <= 0 || H <= 0 || Nq <= 0 || Nk <= 0 || threshold != threshold) return SOL_ERR_INVALID_ARG;
  if (scale != scale || isinf(scale)) return SOL_ERR_INVALID_ARG;
  if (d != 64 && d != 128) return SOL_ERR_UNSUPPORTED_SHAPE;
  if (Nq > 65535 * 8 || (long long)B * H > 65535) return SOL_ERR_UNSUPPORTED_SHAPE;
  const size_t bh = (size_t)B * H;
  if (bh * d * ((size_t)d + 1) > kScratchFloats) return SOL_ERR_SCRATCH_LIMIT;
  sol_status_t s = sol::check_device_arch();
  if (s != SOL_OK) return s;
  float* scratch = nullptr;
  if ((s = scratch_for_current_device(&scratch)) != SOL_OK) return s;
  float* mk = scratch;
  float* cov = scratch + bh * d;
  const float sc = scale > 0.f ? scale : 1.0f / sqrtf((float)d);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  static_key_mean<<<(unsigned)bh, d, 0, st>>>(kc, mk, Nk, d);
  static_key_cov<<<dim3(d / 16, (unsigned)bh), 256, 0, st>>>(kc, mk, cov, Nk, d);
  static_tau<<<dim3((Nq + 7) / 8, (unsigned)bh), 256, 0, st>>>(qbar, mk, cov, mu, sigma, tau, Nq, d, sc, threshold);
  sol::count_launches(3);
  return cudaGetLastError() == cudaSuccess ? SOL_OK : SOL_ERR_CUDA;
}

extern "C" size_t sol_attn_thresholds_static_max_floats(void) { return kScratchFloats; }
