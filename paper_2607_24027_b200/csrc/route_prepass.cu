// Optional routing pre-pass (SOL_ROUTING_PREPASS): the comparison of Eq. (4),
//   s_ij = scale * Qbar_i . KC_j  >  tau_i   (strict),
// evaluated for every (query block, key block) pair before the fused kernel runs, and kept as ONE
// BIT per pair in the caller's mask buffer.  The proxy scores themselves still never reach memory:
// they live in the registers of this kernel for the length of one 64 x 64 tile.  The fused kernel's
// router then only turns the bits into tile records, which takes its shared-memory and
// instruction-issue load off the scheduler it shares with two softmax warps.
//
// Algorithm 1 routes inside the attention loop; this is the same decision taken earlier, so the
// default stays the in-kernel router and this path is an option for low routing densities.
#include "common.cuh"

namespace sol {
namespace {

constexpr int kTile = 64, kChunk = 32;

// grid (ceil(Nk / 64), ceil(Nq / 64), BH), 256 threads; thread (ty, tx) owns rows 4 ty .. 4 ty + 3 and
// columns 4 tx .. 4 tx + 3 of the tile.  mask[bh][i][w]: bit j % 32 of word j / 32 = block j routed.
__global__ void __launch_bounds__(256) mask_prepass_kernel(const float* __restrict__ qbar, const float* __restrict__ kc,
                                                           const float* __restrict__ tau,
                                                           const uint8_t* __restrict__ forced,
                                                           uint32_t* __restrict__ mask, int Nq, int Nk, int d,
                                                           float scale) {
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
  // four decisions per row and thread -> one 32-bit word per row and group of eight threads
  const int words = ceil_div(Nk, 32);
  const int word = j0 / 32 + tx / 8;
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    const int i = i0 + ty * 4 + a;
    const float t = i < Nq ? tau[(size_t)bh * Nq + i] : 0.f;
    uint32_t bits = 0;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int j = j0 + tx * 4 + b;
      bool sel = j < Nk && scale * acc[a][b] > t;
      if (forced && j < Nk && forced[j]) sel = true;
      bits |= (sel ? 1u : 0u) << ((tx % 8) * 4 + b);
    }
    bits |= __shfl_xor_sync(0xffffffffu, bits, 1);
    bits |= __shfl_xor_sync(0xffffffffu, bits, 2);
    bits |= __shfl_xor_sync(0xffffffffu, bits, 4);
    if (tx % 8 == 0 && i < Nq && word < words) mask[((size_t)bh * Nq + i) * words + word] = bits;
  }
}

}  // namespace

cudaError_t launch_route_prepass(const Problem& p, const WsPtrs& ws, const float* tau, uint32_t* mask,
                                 cudaStream_t stream, int* n_launches) {
  const dim3 grid(ceil_div(p.Nk, kTile), ceil_div(p.Nq, kTile), p.BH);
  mask_prepass_kernel<<<grid, 256, 0, stream>>>(ws.qbar, ws.kc, tau, p.forced, mask, p.Nq, p.Nk, p.d, p.scale);
  if (n_launches) *n_launches += 1;
  return cudaGetLastError();
}

}  // namespace sol
