// Sol-Attn fused forward (Algorithm 1), warp-level mma.sync implementation.
//
// One CTA per (batch*head, query block).  The CTA walks the pooled keys in chunks of BLK
// blocks.  For each chunk it (1) scores every block with the proxy s_ij = scale * Qbar_i . KC_j
// (Eq. 3) and compares it with tau_i (Eq. 4) -- the decision lives in shared memory only --,
// (2) runs the approximate branch on the chunk's unselected blocks: the token-to-block tile
// Q_i KC^T feeds the running softmax with multiplicity n_j and the block's mean value
// (Eqs. 9-10 written as a logit bias log n_j), (3) runs exact attention on every selected
// block.  Both branches update one (m, l, acc) held in registers.
//
// This is the portable tensor-core path (m16n8k16 bf16 mma.sync, cp.async staging); it serves
// shapes the tcgen05 kernel does not cover and is the on-device cross-check for it.
#include "common.cuh"

namespace sol {
namespace {

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src));
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(p)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(p)));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

template <int D, int BLK>
struct Smem {
  static constexpr int LD = D + 8;              // padded row (bf16 elements), keeps ldmatrix conflict-free
  __nv_bfloat16 k[BLK][LD];                     // also stages Q at kernel start
  __nv_bfloat16 v[BLK][LD];
  float bias[BLK];                              // per pooled-key column: log2(n_j) or -inf
  float qbar[D];
  int16_t sel_list[BLK];
  int n_sel;
  int any_unselected;
};

// Copy `rows` rows of D bf16 (row_stride elements apart) from global into a padded shared tile;
// rows beyond are zeroed.
template <int D, int BLK, int THREADS>
__device__ __forceinline__ void load_tile(__nv_bfloat16 (*dst)[D + 8], const __nv_bfloat16* src, int rows,
                                          size_t row_stride) {
  constexpr int CPR = D / 8;                    // 16-byte chunks per row
  for (int e = threadIdx.x; e < BLK * CPR; e += THREADS) {
    const int r = e / CPR, c = e % CPR;
    if (r < rows) cp_async16(&dst[r][c * 8], src + (size_t)r * row_stride + c * 8);
    else *reinterpret_cast<uint4*>(&dst[r][c * 8]) = make_uint4(0, 0, 0, 0);
  }
}

template <int D, int BLK>
__global__ void __launch_bounds__(BLK * 2)
fwd_mma_sync_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                    const __nv_bfloat16* __restrict__ v, __nv_bfloat16* __restrict__ out,
                    WsPtrs ws, const float* __restrict__ tau, int32_t* __restrict__ counts,
                    uint32_t* __restrict__ mask_out, const uint8_t* __restrict__ forced, Strides st, int N, int Nq,
                    int Nk, float scale, int mode) {
  constexpr int THREADS = BLK * 2;
  constexpr int WARPS = THREADS / 32;
  constexpr int NT = BLK / 8;                   // score n-tiles (8 key columns each)
  constexpr int KS = D / 16;                    // k-steps of the QK^T contraction
  constexpr int DN = D / 8;                     // output n-tiles (8 channels each)
  extern __shared__ __align__(16) unsigned char smem_raw[];
  auto& sm = *reinterpret_cast<Smem<D, BLK>*>(smem_raw);

  const int i = blockIdx.x, bh = blockIdx.y;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int q_row0 = i * BLK;
  const int q_rows = min(BLK, N - q_row0);
  const float scale_log2 = scale * 1.4426950408889634f;

  // ---- stage Q_i, build its A fragments (kept in registers for the whole kernel)
  const size_t head_base = st.base(bh);          // element offset of (b, h, token 0) in q, k, v, out
  load_tile<D, BLK, THREADS>(sm.k, q + head_base + (size_t)q_row0 * st.row, q_rows, st.row);
  if (mode != SOL_MODE_DENSE)
    for (int c = threadIdx.x; c < D; c += THREADS) sm.qbar[c] = ws.qbar[((size_t)bh * Nq + i) * D + c];
  cp_async_wait_all();
  __syncthreads();
  uint32_t qf[KS][4];
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
    // matrices: (rows 0-7, k 0-7), (rows 8-15, k 0-7), (rows 0-7, k 8-15), (rows 8-15, k 8-15)
    const int m = lane / 8, r = lane % 8;
    ldmatrix_x4(qf[ks], &sm.k[warp * 16 + (m % 2) * 8 + r][ks * 16 + (m / 2) * 8]);
  }
  const float tau_i = (mode == SOL_MODE_DENSE) ? 0.f : tau[(size_t)bh * Nq + i];

  float o_acc[DN][4];
#pragma unroll
  for (int dn = 0; dn < DN; ++dn)
#pragma unroll
    for (int e = 0; e < 4; ++e) o_acc[dn][e] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY};      // running max (log2 domain) of rows lane/4 and lane/4+8
  float l_run[2] = {0.f, 0.f};                  // this thread's share of the running denominator
  int count = 0;

  // One online-softmax step over a staged K-like / V-like tile.
  //   approx = true : columns are pooled keys, bias[col] = log2(n_j) or -inf (selected / padding)
  //   approx = false: columns are tokens, columns >= cols_valid are -inf
  auto process_tile = [&](const __nv_bfloat16* ksrc, const __nv_bfloat16* vsrc, int cols_valid, bool approx) {
    const size_t rs = approx ? (size_t)D : (size_t)st.row;   // pooled operands are dense [Nk][D]
    __syncthreads();                            // everyone is done with the previous tile
    load_tile<D, BLK, THREADS>(sm.k, ksrc, cols_valid, rs);
    load_tile<D, BLK, THREADS>(sm.v, vsrc, cols_valid, rs);
    cp_async_wait_all();
    __syncthreads();

    float s[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) s[nt][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ks += 2) {
        uint32_t kf[4];                         // b0,b1 of k-step ks and of k-step ks+1
        ldmatrix_x4(kf, &sm.k[nt * 8 + lane % 8][ks * 16 + (lane / 8) * 8]);
        mma_bf16(s[nt], qf[ks], kf[0], kf[1]);
        mma_bf16(s[nt], qf[ks + 1], kf[2], kf[3]);
      }
    }
    // logits in the log2 domain, masking
    float tmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int c0 = nt * 8 + (lane % 4) * 2;
      float b0, b1;
      if (approx) { b0 = sm.bias[c0]; b1 = sm.bias[c0 + 1]; }
      else { b0 = (c0 < cols_valid) ? 0.f : -INFINITY; b1 = (c0 + 1 < cols_valid) ? 0.f : -INFINITY; }
      s[nt][0] = fmaf(s[nt][0], scale_log2, b0);
      s[nt][1] = fmaf(s[nt][1], scale_log2, b1);
      s[nt][2] = fmaf(s[nt][2], scale_log2, b0);
      s[nt][3] = fmaf(s[nt][3], scale_log2, b1);
      tmax[0] = fmaxf(tmax[0], fmaxf(s[nt][0], s[nt][1]));
      tmax[1] = fmaxf(tmax[1], fmaxf(s[nt][2], s[nt][3]));
    }
    float alpha[2], m_use[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      tmax[h] = fmaxf(tmax[h], __shfl_xor_sync(0xffffffffu, tmax[h], 1));
      tmax[h] = fmaxf(tmax[h], __shfl_xor_sync(0xffffffffu, tmax[h], 2));
      const float m_new = fmaxf(m_run[h], tmax[h]);
      m_use[h] = (m_new == -INFINITY) ? 0.f : m_new;   // a row that has seen nothing yet
      alpha[h] = fast_exp2(m_run[h] - m_use[h]);       // exp2(-inf) = 0 on the first tile
      m_run[h] = m_new;
      l_run[h] *= alpha[h];
    }
#pragma unroll
    for (int dn = 0; dn < DN; ++dn) {
      o_acc[dn][0] *= alpha[0]; o_acc[dn][1] *= alpha[0];
      o_acc[dn][2] *= alpha[1]; o_acc[dn][3] *= alpha[1];
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      s[nt][0] = fast_exp2(s[nt][0] - m_use[0]);
      s[nt][1] = fast_exp2(s[nt][1] - m_use[0]);
      s[nt][2] = fast_exp2(s[nt][2] - m_use[1]);
      s[nt][3] = fast_exp2(s[nt][3] - m_use[1]);
      l_run[0] += s[nt][0] + s[nt][1];
      l_run[1] += s[nt][2] + s[nt][3];
    }
    // acc += P V
#pragma unroll
    for (int kt = 0; kt < BLK / 16; ++kt) {
      uint32_t pf[4];
      pf[0] = pack_bf16(s[2 * kt][0], s[2 * kt][1]);
      pf[1] = pack_bf16(s[2 * kt][2], s[2 * kt][3]);
      pf[2] = pack_bf16(s[2 * kt + 1][0], s[2 * kt + 1][1]);
      pf[3] = pack_bf16(s[2 * kt + 1][2], s[2 * kt + 1][3]);
#pragma unroll
      for (int dn = 0; dn < DN; dn += 2) {
        uint32_t vf[4];                         // b0,b1 of channel tile dn and of dn+1
        const int m = lane / 8, r = lane % 8;
        ldmatrix_x4_trans(vf, &sm.v[kt * 16 + (m % 2) * 8 + r][(dn + m / 2) * 8]);
        mma_bf16(o_acc[dn], pf, vf[0], vf[1]);
        mma_bf16(o_acc[dn + 1], pf, vf[2], vf[3]);
      }
    }
  };

  // ---- outer loop over chunks of BLK pooled keys
  const int n_chunks = ceil_div(Nk, BLK);
  for (int t = 0; t < n_chunks; ++t) {
    const int j0 = t * BLK;
    __syncthreads();                            // previous chunk's routing state fully consumed
    // routing: proxy score of every block of the chunk against tau_i, decision kept on chip
    for (int jj = warp; jj < BLK; jj += WARPS) {
      const int j = j0 + jj;
      float bias = -INFINITY;
      if (j < Nk) {
        bool sel = true;
        if (mode != SOL_MODE_DENSE) {
          const float* kc = ws.kc + ((size_t)bh * Nk + j) * D;
          float dot = 0.f;
#pragma unroll
          for (int c = 0; c < D / 32; ++c) dot = fmaf(sm.qbar[lane + 32 * c], kc[lane + 32 * c], dot);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
          sel = scale * dot > tau_i;
          if (forced && forced[j]) sel = true;
        }
        if (!sel) bias = log2f((float)min(BLK, N - j * BLK));
      }
      if (lane == 0) sm.bias[jj] = bias;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int n = 0, any_u = 0;
      uint32_t word = 0;
      for (int jj = 0; jj < BLK; ++jj) {
        const int j = j0 + jj;
        const bool valid = j < Nk;
        const bool sel = valid && sm.bias[jj] == -INFINITY;
        if (sel) { sm.sel_list[n++] = (int16_t)jj; word |= 1u << (jj % 32); }
        else if (valid) any_u = 1;
        if (jj % 32 == 31) {
          if (mask_out && (j0 + jj - 31) < Nk)
            mask_out[((size_t)bh * Nq + i) * ceil_div(Nk, 32) + (j0 + jj) / 32] = word;
          word = 0;
        }
      }
      sm.n_sel = n;
      sm.any_unselected = any_u;
      count += n;
    }
    __syncthreads();
    const int n_sel = sm.n_sel;
    if (mode == SOL_MODE_SOL && sm.any_unselected)         // approximate branch, Eqs. (9)-(10)
      process_tile(ws.kcb + ((size_t)bh * Nk + j0) * D, ws.vmb + ((size_t)bh * Nk + j0) * D,
                   min(BLK, Nk - j0), true);
    for (int e = 0; e < n_sel; ++e) {                      // exact branch, inner loop
      const int j = j0 + sm.sel_list[e];
      process_tile(k + head_base + (size_t)j * BLK * st.row, v + head_base + (size_t)j * BLK * st.row,
                   min(BLK, N - j * BLK), false);
    }
  }

  // ---- finalize: O_i = acc / l
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
    l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
  }
  const float inv0 = l_run[0] > 0.f ? 1.f / l_run[0] : 0.f;
  const float inv1 = l_run[1] > 0.f ? 1.f / l_run[1] : 0.f;
  const int r0 = warp * 16 + lane / 4, r1 = r0 + 8;
  __nv_bfloat16* obase = out + head_base + (size_t)q_row0 * st.row;
#pragma unroll
  for (int dn = 0; dn < DN; ++dn) {
    const int c = dn * 8 + (lane % 4) * 2;
    if (r0 < q_rows)
      *reinterpret_cast<uint32_t*>(obase + (size_t)r0 * st.row + c) = pack_bf16(o_acc[dn][0] * inv0, o_acc[dn][1] * inv0);
    if (r1 < q_rows)
      *reinterpret_cast<uint32_t*>(obase + (size_t)r1 * st.row + c) = pack_bf16(o_acc[dn][2] * inv1, o_acc[dn][3] * inv1);
  }
  if (threadIdx.x == 0 && counts) counts[(size_t)bh * Nq + i] = count;
}

template <int D, int BLK>
cudaError_t launch_impl(const Problem& p, const __nv_bfloat16* q, const __nv_bfloat16* k,
                        const __nv_bfloat16* v, __nv_bfloat16* out, const WsPtrs& ws, const float* tau,
                        int32_t* counts, uint32_t* mask_out, cudaStream_t stream) {
  const size_t smem = sizeof(Smem<D, BLK>);
  cudaError_t e = cudaFuncSetAttribute(fwd_mma_sync_kernel<D, BLK>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid(p.Nq, p.BH);
  fwd_mma_sync_kernel<D, BLK><<<grid, BLK * 2, smem, stream>>>(q, k, v, out, ws, tau, counts, mask_out, p.forced,
                                                                p.st, p.N, p.Nq, p.Nk, p.scale, p.mode);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fwd_mma_sync(const Problem& p, const __nv_bfloat16* q, const __nv_bfloat16* k,
                                const __nv_bfloat16* v, __nv_bfloat16* out, const WsPtrs& ws,
                                const float* tau, int32_t* counts, uint32_t* mask_out,
                                cudaStream_t stream, int* n_launches) {
  if (n_launches) *n_launches += 1;
  if (p.d == 128 && p.block_q == 128) return launch_impl<128, 128>(p, q, k, v, out, ws, tau, counts, mask_out, stream);
  if (p.d == 128 && p.block_q == 64) return launch_impl<128, 64>(p, q, k, v, out, ws, tau, counts, mask_out, stream);
  if (p.d == 64 && p.block_q == 128) return launch_impl<64, 128>(p, q, k, v, out, ws, tau, counts, mask_out, stream);
  return launch_impl<64, 64>(p, q, k, v, out, ws, tau, counts, mask_out, stream);
}

}  // namespace sol
