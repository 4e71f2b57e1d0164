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
            const __nv_bfloat16* __restrict__ v, WsPtrs ws, int N, int block_q, int block_k,
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
  const __nv_bfloat16* base = src + ((size_t)bh * N + row0) * D;

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
      x[u] = *reinterpret_cast<const Bf16x8*>(base + (size_t)(row + u * RG) * D + tc * 8);
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
    Bf16x8 x = *reinterpret_cast<const Bf16x8*>(base + (size_t)row * D + tc * 8);
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

// First moment of the pooled keys, m_K = (1/Nk) sum_j KC_j  (Eq. 5).  One CTA per (batch, head),
// thread c owns channel c.
template <int D>
__global__ void __launch_bounds__(D) key_mean_kernel(WsPtrs ws, int Nk) {
  const int bh = blockIdx.x, c = threadIdx.x;
  const float* kc = ws.kc + (size_t)bh * Nk * D;
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
  int j = 0;
  for (; j + 3 < Nk; j += 4) {
    s0 += kc[(size_t)j * D + c];
    s1 += kc[(size_t)(j + 1) * D + c];
    s2 += kc[(size_t)(j + 2) * D + c];
    s3 += kc[(size_t)(j + 3) * D + c];
  }
  for (; j < Nk; ++j) s0 += kc[(size_t)j * D + c];
  ws.mk[(size_t)bh * D + c] = ((s0 + s1) + (s2 + s3)) / (float)Nk;
}

// Centred second moment of the pooled keys,
//   C_K = (1/Nk) sum_j (KC_j - m_K)^T (KC_j - m_K)  =  (1/Nk) sum_j KC_j^T KC_j - m_K^T m_K,
// i.e. the bracket of Eq. (5) with the mu_i^2 term already folded in, which avoids the
// cancellation of the uncentred form in fp32.  Grid (D/16, BH); a CTA of 256 threads owns 16
// rows of C_K, thread (r, cg) owns C_K[r][cg*8 .. cg*8+7].
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
  float acc[CPT];
#pragma unroll
  for (int c = 0; c < CPT; ++c) acc[c] = 0.f;
  for (int j0 = 0; j0 < Nk; j0 += JT) {
    const int nj = min(JT, Nk - j0);
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
  float* cov = ws.covk + ((size_t)bh * D + r) * D + c0;
#pragma unroll
  for (int c = 0; c < CPT; ++c) cov[c] = acc[c] / (float)Nk;
}

// Per-query-block statistics and threshold (Eq. 4, Eq. 5):
//   mu_i = s * Qbar_i . m_K,   sigma_i^2 = s^2 * Qbar_i C_K Qbar_i^T,   tau_i = mu_i + beta sigma_i.
// Grid (ceil(Nq / 64), BH); C_K is staged in shared memory once per CTA; each of the 8 warps
// handles 8 query blocks.
template <int D>
__global__ void __launch_bounds__(256) tau_kernel(WsPtrs ws, int Nq, float scale, float beta) {
  extern __shared__ float cov_s[];               // [D][D+1]
  constexpr int LD = D + 1;
  constexpr int PER = D / 32;                    // channels per lane
  const int bh = blockIdx.y;
  const float* cov = ws.covk + (size_t)bh * D * D;
  for (int e = threadIdx.x; e < D * D; e += 256) cov_s[(e / D) * LD + (e % D)] = cov[e];
  __syncthreads();
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const float* mk = ws.mk + (size_t)bh * D;
  for (int t = 0; t < 8; ++t) {
    const int i = blockIdx.x * 64 + warp * 8 + t;
    if (i >= Nq) break;
    const float* qb = ws.qbar + ((size_t)bh * Nq + i) * D;
    // lane owns rows lane, lane+32, ... of C_K; y_r = sum_c C[r][c] q[c]; quad = sum_r q[r] y_r
    float quad = 0.f, dotm = 0.f;
#pragma unroll
    for (int rr = 0; rr < PER; ++rr) {
      const int r = lane + 32 * rr;
      float y = 0.f;
      for (int c = 0; c < D; ++c) y = fmaf(cov_s[r * LD + c], qb[c], y);
      quad = fmaf(qb[r], y, quad);
      dotm = fmaf(qb[r], mk[r], dotm);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      quad += __shfl_xor_sync(0xffffffffu, quad, o);
      dotm += __shfl_xor_sync(0xffffffffu, dotm, o);
    }
    if (lane == 0) {
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
    pool_kernel<128><<<(unsigned)blocks, kPoolThreads, 0, stream>>>(q, k, v, ws, p.N, p.block_q, p.block_k,
                                                                      p.Nq, p.Nk, first_kind);
  else
    pool_kernel<64><<<(unsigned)blocks, kPoolThreads, 0, stream>>>(q, k, v, ws, p.N, p.block_q, p.block_k,
                                                                     p.Nq, p.Nk, first_kind);
  if (n_launches) *n_launches += 1;
  return cudaGetLastError();
}

template <int D>
static cudaError_t thresholds_impl(const Problem& p, const WsPtrs& ws, cudaStream_t stream, int* n_launches) {
  key_mean_kernel<D><<<p.BH, D, 0, stream>>>(ws, p.Nk);
  key_cov_kernel<D><<<dim3(D / 16, p.BH), 256, 0, stream>>>(ws, p.Nk);
  const size_t smem = sizeof(float) * D * (D + 1);
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(tau_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  tau_kernel<D><<<dim3(ceil_div(p.Nq, 64), p.BH), 256, smem, stream>>>(ws, p.Nq, p.scale, p.beta);
  if (n_launches) *n_launches += 3;
  return cudaGetLastError();
}

cudaError_t launch_thresholds(const Problem& p, const WsPtrs& ws, cudaStream_t stream, int* n_launches) {
  return p.d == 128 ? thresholds_impl<128>(p, ws, stream, n_launches)
                    : thresholds_impl<64>(p, ws, stream, n_launches);
}

}  // namespace sol
