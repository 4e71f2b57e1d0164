// Pre-attention pass of Sol-Attn: block pooling (Eq. 3 and the summed values defined before
// Eq. 9), pooled-key moments (Eq. 5) and per-query-block thresholds (Eq. 4).
//
// The pooling kernel is HBM-bound: it reads q, k and v exactly once with 16-byte loads and
// writes a few MB of pooled vectors.  The moment / threshold kernels touch only pooled data.
#include "common.cuh"

namespace sol {
namespace {

constexpr int kPoolThreads = 256;

struct alignas(16) Bf16x8 { __nv_bfloat162 v[4]; };

// One CTA pools one block of one tensor.  A row of d bf16 is covered by d/8 threads with one
// 16-byte load each; the 256 threads form 256/(d/8) row groups that stride over the block's
// rows; partial sums are combined through shared memory.
//   kind 0: q  -> qbar (mean)
//   kind 1: k  -> kc (mean, fp32) and kcb (mean, bf16)
//   kind 2: v  -> vc (sum, fp32)  and vmb (mean, bf16)
template <int D>
__global__ void __launch_bounds__(kPoolThreads)
pool_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
            const __nv_bfloat16* __restrict__ v, WsPtrs ws, Strides st, int N, int block_q, int block_k,
            int Nq, int Nk, int first_kind) {
  constexpr int TPR = D / 8;                    // threads per row
  constexpr int RG = kPoolThreads / TPR;        // row groups
  __shared__ float partial[RG][D];

  // blockIdx.x enumerates, per (batch, head): Nq query blocks (if q is pooled), Nk key blocks,
  // Nk value blocks.
  const int per_bh = (first_kind == 0 ? Nq : 0) + 2 * Nk;
  const int bh = blockIdx.x / per_bh;
  int r = blockIdx.x - bh * per_bh;
  int kind, blk;
  if (first_kind == 0 && r < Nq) { kind = 0; blk = r; }
  else {
    if (first_kind == 0) r -= Nq;
    if (r < Nk) { kind = 1; blk = r; } else { kind = 2; blk = r - Nk; }
  }
  const int bs = (kind == 0) ? block_q : block_k;
  const __nv_bfloat16* src = (kind == 0) ? q : (kind == 1 ? k : v);
  const int row0 = blk * bs;
  const int nvalid = min(bs, N - row0);
  const __nv_bfloat16* base = src + st.base(bh) + (size_t)row0 * st.row;

  const int tc = threadIdx.x % TPR;             // which 8-channel group of the row
  const int g = threadIdx.x / TPR;              // row group
  float acc[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) acc[c] = 0.f;

  int row = g;
  // four independent 16-byte loads in flight per thread
  for (; row + 3 * RG < nvalid; row += 4 * RG) {
    Bf16x8 x[4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
      x[u] = *reinterpret_cast<const Bf16x8*>(base + (size_t)(row + u * RG) * st.row + tc * 8);
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float2 f = __bfloat1622float2(x[u].v[c]);
        acc[2 * c] += f.x;
        acc[2 * c + 1] += f.y;
      }
  }
  for (; row < nvalid; row += RG) {
    Bf16x8 x = *reinterpret_cast<const Bf16x8*>(base + (size_t)row * st.row + tc * 8);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      float2 f = __bfloat1622float2(x.v[c]);
      acc[2 * c] += f.x;
      acc[2 * c + 1] += f.y;
    }
  }
#pragma unroll
  for (int c = 0; c < 8; ++c) partial[g][tc * 8 + c] = acc[c];
  __syncthreads();

  if (threadIdx.x < D) {
    const int c = threadIdx.x;
    float s = 0.f;
#pragma unroll 8
    for (int gg = 0; gg < RG; ++gg) s += partial[gg][c];
    const float mean = s / (float)nvalid;
    if (kind == 0) {
      ws.qbar[((size_t)bh * Nq + blk) * D + c] = mean;
    } else if (kind == 1) {
      const size_t o = ((size_t)bh * Nk + blk) * D + c;
      ws.kc[o] = mean;
      ws.kcb[o] = __float2bfloat16_rn(mean);
    } else {
      const size_t o = ((size_t)bh * Nk + blk) * D + c;
      ws.vc[o] = s;
      ws.vmb[o] = __float2bfloat16_rn(mean);
    }
  }
}

// First moment of the pooled keys, m_K = (1/Nk) sum_j KC_j  (Eq. 5).  One CTA per (batch, head):
// 4 row groups x D channels, combined through shared memory.
template <int D>
__global__ void __launch_bounds__(4 * D) key_mean_kernel(WsPtrs ws, int Nk) {
  __shared__ float part[4][D];
  const int bh = blockIdx.x, c = threadIdx.x % D, grp = threadIdx.x / D;
  const float* kc = ws.kc + (size_t)bh * Nk * D;
  float s0 = 0.f, s1 = 0.f;
  int j = grp;
  for (; j + 4 < Nk; j += 8) {
    s0 += kc[(size_t)j * D + c];
    s1 += kc[(size_t)(j + 4) * D + c];
  }
  if (j < Nk) s0 += kc[(size_t)j * D + c];
  part[grp][c] = s0 + s1;
  __syncthreads();
  if (grp == 0) ws.mk[(size_t)bh * D + c] = ((part[0][c] + part[1][c]) + (part[2][c] + part[3][c])) / (float)Nk;
}

// Centred second moment of the pooled keys,
//   C_K = (1/Nk) sum_j (KC_j - m_K)^T (KC_j - m_K)  =  (1/Nk) sum_j KC_j^T KC_j - m_K^T m_K,
// i.e. the bracket of Eq. (5) with the mu_i^2 term already folded in, which avoids the
// cancellation of the uncentred form in fp32.  Grid (D/16, BH, key slices); a CTA of 256 threads
// owns 16 rows of C_K for one slice of the pooled keys, thread (r, cg) owns C_K[r][cg*8 ..
// cg*8+7]; every slice writes its own partial matrix (covk holds kCovSlices of them per launch,
// slice-major) and tau_kernel adds them in a fixed order, so the result is bit-stable run to run.

template <int D>
__global__ void __launch_bounds__(256) key_cov_kernel(WsPtrs ws, int Nk) {
  constexpr int ROWS = 16;
  constexpr int CG = 256 / ROWS;                 // column groups per row (16)
  constexpr int CPT = D / CG;                    // columns per thread (8 or 4)
  constexpr int JT = 32;                         // pooled keys staged per step
  __shared__ float xs[JT][D];
  const int bh = blockIdx.y;
  const int r = blockIdx.x * ROWS + threadIdx.x / CG;
  const int c0 = (threadIdx.x % CG) * CPT;
  const float* kc = ws.kc + (size_t)bh * Nk * D;
  const float* mk = ws.mk + (size_t)bh * D;
  const int per_slice = ceil_div(Nk, kCovSlices);
  const int j_begin = blockIdx.z * per_slice, j_end = min(Nk, j_begin + per_slice);
  float acc[CPT];
#pragma unroll
  for (int c = 0; c < CPT; ++c) acc[c] = 0.f;
  for (int j0 = j_begin; j0 < j_end; j0 += JT) {
    const int nj = min(JT, j_end - j0);
    for (int e = threadIdx.x; e < nj * D; e += 256) {
      const int jj = e / D, c = e % D;
      xs[jj][c] = kc[(size_t)(j0 + jj) * D + c] - mk[c];
    }
    __syncthreads();
    for (int jj = 0; jj < nj; ++jj) {
      const float xr = xs[jj][r];
#pragma unroll
      for (int c = 0; c < CPT; ++c) acc[c] = fmaf(xr, xs[jj][c0 + c], acc[c]);
    }
    __syncthreads();
  }
  float* cov = ws.covk + (((size_t)blockIdx.z * gridDim.y + bh) * D + r) * D + c0;
#pragma unroll
  for (int c = 0; c < CPT; ++c) cov[c] = acc[c] / (float)Nk;
}

// Per-query-block statistics and threshold (Eq. 4, Eq. 5):
//   mu_i = s * Qbar_i . m_K,   sigma_i^2 = s^2 * Qbar_i C_K Qbar_i^T,   tau_i = mu_i + beta sigma_i.
// Grid (ceil(Nq / 64), BH).  A CTA stages C_K and 64 pooled queries in shared memory and forms
// Y = Qbar C_K as a register-tiled product (thread (rg, cg): 4 query blocks x 8 channels); the
// quadratic form is the row sum of Y o Qbar, reduced over the 16 threads of a query-block group.
template <int D>
__global__ void __launch_bounds__(256) tau_kernel(WsPtrs ws, int Nq, float scale, float beta) {
  extern __shared__ float smem_f[];
  constexpr int QT = 64;                         // query blocks per CTA
  constexpr int CPT = D / 16;                    // channels per thread (8 or 4)
  float* cov_s = smem_f;                         // [D][D]
  float* q_s = smem_f + D * D;                   // [QT][D + 1]
  constexpr int QLD = D + 1;
  const int bh = blockIdx.y, i0 = blockIdx.x * QT;
  const size_t slice_stride = (size_t)gridDim.y * D * D;
  const float* cov = ws.covk + (size_t)bh * D * D;
  for (int e = threadIdx.x; e < D * D / 4; e += 256) {
    float4 a = reinterpret_cast<const float4*>(cov)[e];
#pragma unroll
    for (int sl = 1; sl < kCovSlices; ++sl) {
      const float4 b = reinterpret_cast<const float4*>(cov + sl * slice_stride)[e];
      a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
    }
    reinterpret_cast<float4*>(cov_s)[e] = a;
  }
  for (int e = threadIdx.x; e < QT * D; e += 256) {
    const int rq = e / D, c = e % D;
    q_s[rq * QLD + c] = (i0 + rq < Nq) ? ws.qbar[((size_t)bh * Nq + i0 + rq) * D + c] : 0.f;
  }
  __syncthreads();
  const int rg = threadIdx.x / 16, cg = threadIdx.x % 16;
  const int c0 = cg * CPT;
  float y[4][CPT];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int c = 0; c < CPT; ++c) y[a][c] = 0.f;
  for (int k = 0; k < D; ++k) {
    float qa[4], cb[CPT];
#pragma unroll
    for (int a = 0; a < 4; ++a) qa[a] = q_s[(rg * 4 + a) * QLD + k];
#pragma unroll
    for (int c = 0; c < CPT; ++c) cb[c] = cov_s[k * D + c0 + c];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int c = 0; c < CPT; ++c) y[a][c] = fmaf(qa[a], cb[c], y[a][c]);
  }
  const float* mk = ws.mk + (size_t)bh * D;
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    float quad = 0.f, dotm = 0.f;
#pragma unroll
    for (int c = 0; c < CPT; ++c) {
      const float qv = q_s[(rg * 4 + a) * QLD + c0 + c];
      quad = fmaf(y[a][c], qv, quad);
      dotm = fmaf(qv, mk[c0 + c], dotm);
    }
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) {
      quad += __shfl_xor_sync(0xffffffffu, quad, o);
      dotm += __shfl_xor_sync(0xffffffffu, dotm, o);
    }
    const int i = i0 + rg * 4 + a;
    if (cg == 0 && i < Nq) {
      const float mu = scale * dotm;
      const float sigma = scale * sqrtf(fmaxf(quad, 0.f));
      float tau;
      if (isinf(beta)) tau = beta;               // +inf: route nothing, -inf: route everything
      else tau = fmaf(beta, sigma, mu);
      const size_t o = (size_t)bh * Nq + i;
      ws.mu[o] = mu;
      ws.sigma[o] = sigma;
      ws.tau[o] = tau;
    }
  }
}

}  // namespace

cudaError_t launch_pool(const Problem& p, const __nv_bfloat16* q, const __nv_bfloat16* k,
                        const __nv_bfloat16* v, const WsPtrs& ws, cudaStream_t stream, int* n_launches) {
  const int first_kind = q ? 0 : 1;
  const long long blocks = (long long)p.BH * ((q ? p.Nq : 0) + 2LL * p.Nk);
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  if (p.d == 128)
    pool_kernel<128><<<(unsigned)blocks, kPoolThreads, 0, stream>>>(q, k, v, ws, p.st, p.N, p.block_q, p.block_k,
                                                                      p.Nq, p.Nk, first_kind);
  else
    pool_kernel<64><<<(unsigned)blocks, kPoolThreads, 0, stream>>>(q, k, v, ws, p.st, p.N, p.block_q, p.block_k,
                                                                     p.Nq, p.Nk, first_kind);
  if (n_launches) *n_launches += 1;
  return cudaGetLastError();
}

// Diagonal estimator (appendix, Eq. appendix_diagonal_threshold): only the per-channel variance of
// the pooled keys is kept, v_K = mean_j KC_j o KC_j - m_K o m_K (computed in centred form), and
// sigma_i^2 = s^2 (Qbar_i o Qbar_i) . v_K.  One CTA per (batch, head) writes m_K and v_K (v_K goes
// to the first D floats of the head's second-moment area).
template <int D>
__global__ void __launch_bounds__(4 * D) key_diag_kernel(WsPtrs ws, int Nk) {
  __shared__ float part[4][D];
  __shared__ float mean_s[D];
  const int bh = blockIdx.x, c = threadIdx.x % D, grp = threadIdx.x / D;
  const float* kc = ws.kc + (size_t)bh * Nk * D;
  float s = 0.f;
  for (int j = grp; j < Nk; j += 4) s += kc[(size_t)j * D + c];
  part[grp][c] = s;
  __syncthreads();
  if (grp == 0) mean_s[c] = ((part[0][c] + part[1][c]) + (part[2][c] + part[3][c])) / (float)Nk;
  __syncthreads();
  const float m = mean_s[c];
  float v = 0.f;
  for (int j = grp; j < Nk; j += 4) {
    const float x = kc[(size_t)j * D + c] - m;
    v = fmaf(x, x, v);
  }
  __syncthreads();
  part[grp][c] = v;
  __syncthreads();
  if (grp == 0) {
    ws.mk[(size_t)bh * D + c] = m;
    ws.covk[(size_t)bh * D * D + c] = ((part[0][c] + part[1][c]) + (part[2][c] + part[3][c])) / (float)Nk;
  }
}

// One warp per query block: mu_i, sigma_i (diagonal form), tau_i.
template <int D>
__global__ void __launch_bounds__(256) tau_diag_kernel(WsPtrs ws, int Nq, float scale, float beta) {
  const int bh = blockIdx.y;
  const int i = blockIdx.x * 8 + threadIdx.x / 32, lane = threadIdx.x % 32;
  if (i >= Nq) return;
  const float* qb = ws.qbar + ((size_t)bh * Nq + i) * D;
  const float* mk = ws.mk + (size_t)bh * D;
  const float* vk = ws.covk + (size_t)bh * D * D;
  float quad = 0.f, dotm = 0.f;
#pragma unroll
  for (int c = lane; c < D; c += 32) {
    const float qv = qb[c];
    quad = fmaf(qv * qv, vk[c], quad);
    dotm = fmaf(qv, mk[c], dotm);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    quad += __shfl_xor_sync(0xffffffffu, quad, o);
    dotm += __shfl_xor_sync(0xffffffffu, dotm, o);
  }
  if (lane == 0) {
    const float mu = scale * dotm;
    const float sigma = scale * sqrtf(fmaxf(quad, 0.f));
    const size_t o = (size_t)bh * Nq + i;
    ws.mu[o] = mu;
    ws.sigma[o] = sigma;
    ws.tau[o] = isinf(beta) ? beta : fmaf(beta, sigma, mu);
  }
}

template <int D>
static cudaError_t thresholds_impl(const Problem& p, const WsPtrs& ws, cudaStream_t stream, int* n_launches) {
  if (p.estimator == SOL_EST_DIAGONAL) {
    key_diag_kernel<D><<<p.BH, 4 * D, 0, stream>>>(ws, p.Nk);
    tau_diag_kernel<D><<<dim3(ceil_div(p.Nq, 8), p.BH), 256, 0, stream>>>(ws, p.Nq, p.scale, p.beta);
    if (n_launches) *n_launches += 2;
    return cudaGetLastError();
  }
  key_mean_kernel<D><<<p.BH, 4 * D, 0, stream>>>(ws, p.Nk);
  key_cov_kernel<D><<<dim3(D / 16, p.BH, kCovSlices), 256, 0, stream>>>(ws, p.Nk);
  const size_t smem = sizeof(float) * (D * D + 64 * (D + 1));
  cudaError_t e = cudaFuncSetAttribute(tau_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  tau_kernel<D><<<dim3(ceil_div(p.Nq, 64), p.BH), 256, smem, stream>>>(ws, p.Nq, p.scale, p.beta);
  if (n_launches) *n_launches += 3;
  return cudaGetLastError();
}

cudaError_t launch_thresholds(const Problem& p, const WsPtrs& ws, cudaStream_t stream, int* n_launches) {
  return p.d == 128 ? thresholds_impl<128>(p, ws, stream, n_launches)
                    : thresholds_impl<64>(p, ws, stream, n_launches);
}

}  // namespace sol
