// sol_attn_route_materialized: the two routing baselines the paper measures its on-the-fly
// thresholding against (introduction, limitation L1; routing-latency figure): the block proxy map
// s_ij = scale * Qbar_i . KC_j (Eq. 3) is WRITTEN TO MEMORY, every row is sorted, and
//   top-k keeps the k highest-scoring key blocks of each query block,
//   top-p keeps blocks in descending order until their share of the row's softmax mass reaches p.
// The result is handed back as routing indices, counts and an equivalent per-row cutoff tau (the
// midpoint between the last kept and the first dropped score), which the fused kernel accepts as
// its threshold array -- so both policies can also drive the single-pass kernel.
#include <math.h>

#include "common.cuh"

namespace {

constexpr int kMaxRow = 8192;          // longest proxy row the in-shared-memory sort takes
constexpr int kTile = 64, kChunk = 32;

// map[bh][i][j] = scale * sum_c qbar[bh][i][c] * kc[bh][j][c]; grid (ceil(Nk/64), ceil(Nq/64), BH),
// 256 threads, each owns a 4 x 4 patch of a 64 x 64 tile.
__global__ void __launch_bounds__(256) proxy_map_kernel(const float* __restrict__ qbar, const float* __restrict__ kc,
                                                        float* __restrict__ map, int Nq, int Nk, int d, float scale) {
  __shared__ float qs[kTile][kChunk + 1];
  __shared__ float ks[kTile][kChunk + 1];
  const int bh = blockIdx.z, i0 = blockIdx.y * kTile, j0 = blockIdx.x * kTile;
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
  const float* qh = qbar + (size_t)bh * Nq * d;
  const float* kh = kc + (size_t)bh * Nk * d;
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
  for (int c0 = 0; c0 < d; c0 += kChunk) {
    for (int e = threadIdx.x; e < kTile * kChunk; e += 256) {
      const int r = e / kChunk, c = e % kChunk;
      qs[r][c] = (i0 + r < Nq) ? qh[(size_t)(i0 + r) * d + c0 + c] : 0.f;
      ks[r][c] = (j0 + r < Nk) ? kh[(size_t)(j0 + r) * d + c0 + c] : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int c = 0; c < kChunk; ++c) {
      float qv[4], kv[4];
#pragma unroll
      for (int a = 0; a < 4; ++a) { qv[a] = qs[ty * 4 + a][c]; kv[a] = ks[tx * 4 + a][c]; }
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(qv[a], kv[b], acc[a][b]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    const int i = i0 + ty * 4 + a;
    if (i >= Nq) continue;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int j = j0 + tx * 4 + b;
      if (j < Nk) map[((size_t)bh * Nq + i) * Nk + j] = scale * acc[a][b];
    }
  }
}

// true when (va, ia) sorts before (vb, ib): higher score first, lower block index on ties
__device__ __forceinline__ bool before(float va, int ia, float vb, int ib) {
  return va > vb || (va == vb && ia < ib);
}

// One CTA per proxy row: read it back from memory, sort it, apply the policy.
__global__ void __launch_bounds__(256) row_select_kernel(const float* __restrict__ map, int Nq, int Nk, int npad,
                                                         int policy, float param, int32_t* __restrict__ order,
                                                         float* __restrict__ tau, int32_t* __restrict__ counts) {
  extern __shared__ unsigned char smem_raw[];
  float* val = reinterpret_cast<float*>(smem_raw);
  int* idx = reinterpret_cast<int*>(val + npad);
  __shared__ double part[256];
  __shared__ double total_s;
  __shared__ int cut;
  const int i = blockIdx.x, bh = blockIdx.y;
  const size_t row = (size_t)bh * Nq + i;
  const float* src = map + row * Nk;
  for (int j = threadIdx.x; j < npad; j += 256) {
    val[j] = j < Nk ? src[j] : -INFINITY;
    idx[j] = j < Nk ? j : 0x7fffffff;
  }
  __syncthreads();
  // bitonic sort, descending
  for (int size = 2; size <= npad; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int t = threadIdx.x; t < npad / 2; t += 256) {
        const int lo = 2 * t - (t & (stride - 1));
        const int hi = lo + stride;
        const bool descending = (lo & size) == 0;
        const float va = val[lo], vb = val[hi];
        const int ia = idx[lo], ib = idx[hi];
        if (before(vb, ib, va, ia) == descending) {
          val[lo] = vb; val[hi] = va;
          idx[lo] = ib; idx[hi] = ia;
        }
      }
      __syncthreads();
    }
  }
  int c;
  if (policy == SOL_ROUTE_TOPK) {
    c = min(max((int)param, 0), Nk);
  } else {
    // share of the row's softmax mass held by the first c blocks; double so that the running sum
    // is not what decides a close call
    const int per = (npad + 255) / 256;
    const int j0 = threadIdx.x * per, j1 = min(j0 + per, Nk);
    const float top = val[0];
    double local = 0.0;
    for (int j = j0; j < j1; ++j) local += exp((double)val[j] - (double)top);
    part[threadIdx.x] = local;
    if (threadIdx.x == 0) cut = Nk;
    __syncthreads();
    if (threadIdx.x == 0) {
      double run = 0.0;
      for (int t = 0; t < 256; ++t) { const double x = part[t]; part[t] = run; run += x; }   // exclusive scan
      total_s = run;
    }
    __syncthreads();
    const double need = (double)param * total_s;
    double run = part[threadIdx.x];
    int first = Nk;
    // the first c with mass(c) >= need; mass(c) = sum of the first c blocks
    if (run < need) {
      for (int j = j0; j < j1; ++j) {
        run += exp((double)val[j] - (double)top);
        if (run >= need) { first = j + 1; break; }
      }
    }
    if (first < Nk) atomicMin(&cut, first);
    __syncthreads();
    c = cut;
    if (need <= 0.0) c = 0;
  }
  if (order)
    for (int j = threadIdx.x; j < Nk; j += 256) order[row * Nk + j] = idx[j];
  if (threadIdx.x == 0) {
    float t;
    if (c <= 0) t = INFINITY;
    else if (c >= Nk) t = -INFINITY;
    else t = 0.5f * (val[c - 1] + val[c]);
    tau[row] = t;
    if (counts) counts[row] = c;
  }
}

}  // namespace

extern "C" sol_status_t sol_attn_route_materialized(const float* qbar, const float* kc, int B, int H, int Nq, int Nk,
                                                    int d, float scale, int policy, float param, float* proxy_map,
                                                    int32_t* order, float* tau, int32_t* counts, sol_stream_t stream) {
  if (!qbar || !kc || !proxy_map || !tau) return SOL_ERR_INVALID_ARG;
  if (B <= 0 || H <= 0 || Nq <= 0 || Nk <= 0 || d <= 0 || param != param) return SOL_ERR_INVALID_ARG;
  if (policy != SOL_ROUTE_TOPK && policy != SOL_ROUTE_TOPP) return SOL_ERR_INVALID_ARG;
  if (policy == SOL_ROUTE_TOPP && (param < 0.f || param > 1.f)) return SOL_ERR_INVALID_ARG;
  if (d % 32 != 0 || Nk > kMaxRow || Nq > 65535 * kTile || (long long)B * H > 65535) return SOL_ERR_UNSUPPORTED_SHAPE;
  const int BH = B * H;
  const float sc = scale > 0.f ? scale : 1.0f / sqrtf((float)d);
  int npad = 2;
  while (npad < Nk) npad <<= 1;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  proxy_map_kernel<<<dim3((Nk + kTile - 1) / kTile, (Nq + kTile - 1) / kTile, BH), 256, 0, st>>>(qbar, kc, proxy_map,
                                                                                                  Nq, Nk, d, sc);
  const size_t smem = (size_t)npad * 8;
  if (cudaFuncSetAttribute(row_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return SOL_ERR_CUDA;
  row_select_kernel<<<dim3(Nq, BH), 256, smem, st>>>(proxy_map, Nq, Nk, npad, policy, param, order, tau, counts);
  sol::count_launches(2);
  return cudaGetLastError() == cudaSuccess ? SOL_OK : SOL_ERR_CUDA;
}
