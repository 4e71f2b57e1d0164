// Shared declarations of the Sol-Attn CUDA path: problem description, workspace layout,
// launch prototypes.  Nothing here is used by the CPU oracle.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "sol_attn.h"

namespace sol {

constexpr int kStatusWords = 16;      // int32 words at the start of the workspace
constexpr int kStatusDevice = 0;      // word 0: device status (0 ok, SOL_ERR_DEVICE_TIMEOUT ...)
constexpr int kStatusDetail = 1;      // word 1: where a bounded wait gave up (debug aid)
constexpr int kStatusTileCounter = 2; // word 2: persistent-kernel work counter
constexpr int kCovSlices = 4;         // partial second-moment matrices per (batch, head)

__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Where element (b, h, n, 0) of q, k, v and out sits (all four share one layout): element strides
// between consecutive tokens, heads and batches.  A token's d channels are always contiguous.
struct Strides {
  long long row, head, batch;
  int H;
  __host__ __device__ size_t base(int bh) const {
    const int b = bh / H;
    return (size_t)b * (size_t)batch + (size_t)(bh - b * H) * (size_t)head;
  }
};

// One attention problem and where its pre-attention results live.
struct Problem {
  int B, H, N, d, block_q, block_k;
  int BH, Nq, Nk;
  float scale;       // logit scale
  float beta;        // standardized cutoff of Eq. (4)
  int mode;          // SOL_MODE_*
  int estimator;     // SOL_EST_*: how sigma_i is obtained
  const uint8_t* forced;   // device [Nk] or null: key blocks that always go to the exact branch
  Strides st;              // SOL_LAYOUT_*: strides of q, k, v, out
  int routing;             // SOL_ROUTING_*: where the comparison of Eq. (4) is evaluated
};

// Byte offsets into the workspace (all multiples of 1024).
struct WsLayout {
  size_t status;  // int32[kStatusWords]
  size_t qbar;    // fp32 [BH][Nq][d]   mean of each query block        (Eq. 3)
  size_t kc;      // fp32 [BH][Nk][d]   mean of each key block          (Eq. 3)
  size_t vc;      // fp32 [BH][Nk][d]   sum of each value block         (before Eq. 9)
  size_t kcb;     // bf16 [BH][Nk][d]   KC rounded, MMA operand of the approximate branch
  size_t vmb;     // bf16 [BH][Nk][d]   VC / n_j rounded, MMA operand of the approximate branch
  size_t mk;      // fp32 [BH][d]       first moment of the pooled keys (Eq. 5)
  size_t covk;    // fp32 [kCovSlices][BH][d][d]  partial centred second moments of the pooled keys (Eq. 5)
  size_t mu, sigma, tau;  // fp32 [BH][Nq] each (Eq. 4)
  size_t total;
};

inline WsLayout make_layout(int BH, int Nq, int Nk, int d) {
  WsLayout w{};
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return o; };
  w.status = take(sizeof(int32_t) * kStatusWords);
  w.qbar = take(sizeof(float) * (size_t)BH * Nq * d);
  w.kc = take(sizeof(float) * (size_t)BH * Nk * d);
  w.vc = take(sizeof(float) * (size_t)BH * Nk * d);
  w.kcb = take(2 * (size_t)BH * Nk * d);
  w.vmb = take(2 * (size_t)BH * Nk * d);
  w.mk = take(sizeof(float) * (size_t)BH * d);
  w.covk = take(sizeof(float) * (size_t)kCovSlices * BH * d * d);
  w.mu = take(sizeof(float) * (size_t)BH * Nq);
  w.sigma = take(sizeof(float) * (size_t)BH * Nq);
  w.tau = take(sizeof(float) * (size_t)BH * Nq);
  w.total = off;
  return w;
}

// Device pointers handed to the kernels.
struct WsPtrs {
  int32_t* status;
  float *qbar, *kc, *vc;
  __nv_bfloat16 *kcb, *vmb;
  float *mk, *covk, *mu, *sigma, *tau;
};

inline WsPtrs make_ptrs(void* base, const WsLayout& w) {
  char* b = static_cast<char*>(base);
  WsPtrs p;
  p.status = reinterpret_cast<int32_t*>(b + w.status);
  p.qbar = reinterpret_cast<float*>(b + w.qbar);
  p.kc = reinterpret_cast<float*>(b + w.kc);
  p.vc = reinterpret_cast<float*>(b + w.vc);
  p.kcb = reinterpret_cast<__nv_bfloat16*>(b + w.kcb);
  p.vmb = reinterpret_cast<__nv_bfloat16*>(b + w.vmb);
  p.mk = reinterpret_cast<float*>(b + w.mk);
  p.covk = reinterpret_cast<float*>(b + w.covk);
  p.mu = reinterpret_cast<float*>(b + w.mu);
  p.sigma = reinterpret_cast<float*>(b + w.sigma);
  p.tau = reinterpret_cast<float*>(b + w.tau);
  return p;
}

// Host-side helpers shared by the files that implement entry points (defined in api.cu).
void count_launches(int n);            // adds to the library's launch counter (sol_attn_launch_count)
sol_status_t check_device_arch();      // SOL_OK on compute capability 10.x, else SOL_ERR_UNSUPPORTED_ARCH

// ---- launchers (each returns the cudaError_t of its launches; all work goes to `stream`) ----

// Pooling pre-pass: Qbar, KC, VC (+ bf16 operand copies).  q may be null.
cudaError_t launch_pool(const Problem& p, const __nv_bfloat16* q, const __nv_bfloat16* k,
                        const __nv_bfloat16* v, const WsPtrs& ws, cudaStream_t stream, int* n_launches);

// Pooled-key moments (Eq. 5) and per-query-block mu, sigma, tau (Eq. 4).
cudaError_t launch_thresholds(const Problem& p, const WsPtrs& ws, cudaStream_t stream, int* n_launches);

// Routing pre-pass (SOL_ROUTING_PREPASS): one decision bit per (query block, key block) into `mask`.
cudaError_t launch_route_prepass(const Problem& p, const WsPtrs& ws, const float* tau, uint32_t* mask,
                                 cudaStream_t stream, int* n_launches);

// Fused forward, warp-level mma.sync implementation (all supported shapes).
cudaError_t launch_fwd_mma_sync(const Problem& p, const __nv_bfloat16* q, const __nv_bfloat16* k,
                                const __nv_bfloat16* v, __nv_bfloat16* out, const WsPtrs& ws,
                                const float* tau, int32_t* counts, uint32_t* mask_out,
                                cudaStream_t stream, int* n_launches);

// Fused forward, TMA + tcgen05 + TMEM implementation (d in {64, 128}, block_q = block_k in {64, 128}).
bool fwd_sm100_supports(const Problem& p);
// Test hook: SM clocks after which the kernel's bounded waits give up (<= 0: the default) and the tile
// whose P V completion signal each CTA leaves out (< 0: none); applies to the following launches.
void fwd_sm100_set_wait(long long wait_cycles, int withhold_tile);
cudaError_t launch_fwd_sm100(const Problem& p, const __nv_bfloat16* q, const __nv_bfloat16* k,
                             const __nv_bfloat16* v, __nv_bfloat16* out, const WsPtrs& ws,
                             const float* tau, int32_t* counts, uint32_t* mask_out,
                             cudaStream_t stream, int* n_launches);

}  // namespace sol
