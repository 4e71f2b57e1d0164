// Two microbenchmarks behind the fused kernel's design notes (timing only; built and run by
// `python -m paper_2607_24027_b200.softmax_probe`, not part of libsol_attn.so):
//
//  run_probe_softmax   the softmax warps' inner loop in isolation -- TMEM load of a score row piece,
//                      maximum, exp2 (special-function unit, or a cubic on the FMA pipes for some of
//                      the element pairs), row sum, bf16 packing, TMEM store -- with 4 or 8 warps on an
//                      otherwise idle SM: cycles per tile.
//  run_probe_handover  what passing an mbarrier between two threads of different warps costs (plain
//                      arrive, or eight MMAs + tcgen05.commit), on an idle SM and beside eight warps
//                      that keep the special-function unit and the TMEM path busy: cycles per round trip.
#include <cstdio>

#include <cuda_bf16.h>

#include "ptx_sm100.cuh"

using namespace sol::ptx;

namespace {

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// exp2 of a pair on the FMA pipes: j = round(x) with the 1.5 * 2^23 trick, a cubic for 2^f on
// f = x - j in [-0.5, 0.5] (minimax in the relative error, 7.5e-5), j added into the exponent
// field with one integer multiply-add.
__device__ __forceinline__ float2 exp2_cubic(float2 x) {
  x.x = fmaxf(x.x, -125.f);
  x.y = fmaxf(x.y, -125.f);
  const float2 magic = make_float2(12582912.f, 12582912.f), neg_magic = make_float2(-12582912.f, -12582912.f);
  const float2 r = __fadd2_rn(x, magic);
  const float2 j = __fadd2_rn(r, neg_magic);
  const float2 f = __ffma2_rn(j, make_float2(-1.f, -1.f), x);
  float2 pl = __ffma2_rn(f, make_float2(0.0551716648f, 0.0551716648f), make_float2(0.2426111251f, 0.2426111251f));
  pl = __ffma2_rn(pl, f, make_float2(0.6932609677f, 0.6932609677f));
  pl = __ffma2_rn(pl, f, make_float2(0.9999280572f, 0.9999280572f));
  int ex, ey;
  asm("mad.lo.s32 %0, %1, %2, %3;" : "=r"(ex) : "r"(__float_as_int(r.x)), "r"(0x800000), "r"(__float_as_int(pl.x)));
  asm("mad.lo.s32 %0, %1, %2, %3;" : "=r"(ey) : "r"(__float_as_int(r.y)), "r"(0x800000), "r"(__float_as_int(pl.y)));
  return make_float2(__int_as_float(ex), __int_as_float(ey));
}

// MASK: bit i set = element pair i (mod 8) of the row takes the cubic; NOEX: no exp2 at all;
// MAX3: 3-input maximum; COLS: score columns per thread.
template <int MASK, int NOEX, int MAX3, int COLS>
__global__ void __launch_bounds__(384, 1) probe_softmax(long long* out, int iters, float sl2, int active_warps) {
  __shared__ uint32_t tmem_base_s;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  if (warp == 0) { tmem_alloc(&tmem_base_s, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  if (warp < active_warps) {
    const uint32_t t_s = tmem + ((uint32_t)((warp % 4) * 32) << 16) + (warp / 4) * COLS;
    uint32_t sr[COLS];
#pragma unroll
    for (int c = 0; c < COLS; ++c) sr[c] = __float_as_uint(-1.0f - 0.01f * c);
#pragma unroll
    for (int c = 0; c < COLS; c += 32) tmem_st_32x32b_x32(t_s + c, *reinterpret_cast<uint32_t(*)[32]>(&sr[c]));
    tmem_st_wait();
    float m_used = 0.f, l = 0.f;
    const long long t0 = clock64();
#pragma unroll 1
    for (int it = 0; it < iters; ++it) {
#pragma unroll
      for (int c = 0; c < COLS; c += 32) tmem_ld_32x32b_x32(t_s + c, *reinterpret_cast<uint32_t(*)[32]>(&sr[c]));
      tmem_ld_wait();
      constexpr int kQ = COLS / 4;
      float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
      if (MAX3) {
#pragma unroll
        for (int c = 0; c < kQ; c += 2) {
          m0 = max3(m0, __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]));
          m1 = max3(m1, __uint_as_float(sr[kQ + c]), __uint_as_float(sr[kQ + c + 1]));
          m2 = max3(m2, __uint_as_float(sr[2 * kQ + c]), __uint_as_float(sr[2 * kQ + c + 1]));
          m3 = max3(m3, __uint_as_float(sr[3 * kQ + c]), __uint_as_float(sr[3 * kQ + c + 1]));
        }
      } else {
#pragma unroll
        for (int c = 0; c < kQ; ++c) {
          m0 = fmaxf(m0, __uint_as_float(sr[c]));
          m1 = fmaxf(m1, __uint_as_float(sr[kQ + c]));
          m2 = fmaxf(m2, __uint_as_float(sr[2 * kQ + c]));
          m3 = fmaxf(m3, __uint_as_float(sr[3 * kQ + c]));
        }
      }
      const float mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)) * sl2;
      if (__any_sync(0xffffffffu, mx > m_used + 8.f)) { m_used = fmaxf(m_used, mx); l *= 0.5f; }
      const float nm = -m_used;
      const float2 sl2_2 = make_float2(sl2, sl2), nm2 = make_float2(nm, nm);
      float2 s_a = make_float2(0.f, 0.f), s_b = make_float2(0.f, 0.f);
#pragma unroll
      for (int c = 0; c < COLS; c += 4) {
        const float2 xa = __ffma2_rn(make_float2(__uint_as_float(sr[c]), __uint_as_float(sr[c + 1])), sl2_2, nm2);
        const float2 xb = __ffma2_rn(make_float2(__uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3])), sl2_2, nm2);
        const bool pa = (MASK >> ((c / 2) % 8)) & 1, pb = (MASK >> ((c / 2 + 1) % 8)) & 1;
        const float2 ea = NOEX ? xa : pa ? exp2_cubic(xa) : make_float2(ex2(xa.x), ex2(xa.y));
        const float2 eb = NOEX ? xb : pb ? exp2_cubic(xb) : make_float2(ex2(xb.x), ex2(xb.y));
        s_a = __fadd2_rn(s_a, ea);
        s_b = __fadd2_rn(s_b, eb);
        __nv_bfloat162 lo = __floats2bfloat162_rn(ea.x, ea.y);
        __nv_bfloat162 hi = __floats2bfloat162_rn(eb.x, eb.y);
        sr[c / 2] = *reinterpret_cast<uint32_t*>(&lo);
        sr[c / 2 + 1] = *reinterpret_cast<uint32_t*>(&hi);
      }
      {
        const float2 tt = __fadd2_rn(s_a, s_b);
        l += tt.x + tt.y;
      }
#pragma unroll
      for (int c = 0; c < COLS / 2; c += 32) tmem_st_32x32b_x32(t_s + 256 + c, *reinterpret_cast<uint32_t(*)[32]>(&sr[c]));
      tmem_st_wait();
    }
    const long long t1 = clock64();
    if (lane == 0) out[blockIdx.x * 16 + warp] = t1 - t0;
    if (l == 123.456f) out[0] = sr[5] + sr[COLS / 2 + 3];   // keeps the arithmetic alive
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

template <int MASK, int NOEX, int MAX3>
int launch_softmax(long long* out, int cols, int iters, int grid, int active) {
  if (cols == 64) probe_softmax<MASK, NOEX, MAX3, 64><<<grid, 384>>>(out, iters, 0.1275f, active);
  else probe_softmax<MASK, NOEX, MAX3, 128><<<grid, 384>>>(out, iters, 0.1275f, active);
  const cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) { printf("cuda error %s\n", cudaGetErrorString(e)); return -2; }
  return 0;
}

}  // namespace

// out: int64[16 * grid], cycles of each active warp of each CTA.  variant: 0 as in the kernel, 1 no exp2,
// 2 three-input maximum, 3 / 4 / 5 / 6 cubic exp2 on 25 / 37.5 / 50 / 100 % of the pairs.  cols: 64 or 128.
extern "C" int run_probe_softmax(long long* out, int variant, int cols, int iters, int grid, int active_warps) {
  if (cols != 64 && cols != 128) return -3;
  switch (variant) {
    case 0: return launch_softmax<0x00, 0, 0>(out, cols, iters, grid, active_warps);
    case 1: return launch_softmax<0x00, 1, 0>(out, cols, iters, grid, active_warps);
    case 2: return launch_softmax<0x00, 0, 1>(out, cols, iters, grid, active_warps);
    case 3: return launch_softmax<0x88, 0, 0>(out, cols, iters, grid, active_warps);
    case 4: return launch_softmax<0xa8, 0, 0>(out, cols, iters, grid, active_warps);
    case 5: return launch_softmax<0xaa, 0, 0>(out, cols, iters, grid, active_warps);
    case 6: return launch_softmax<0xff, 0, 0>(out, cols, iters, grid, active_warps);
    default: return -3;
  }
}

// ------------------------------------------------------------------------------------------------
namespace {

__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
  return ok != 0;
}
constexpr int kSpinLimit = 1000000;
__device__ __forceinline__ bool spin_test(uint64_t* bar, uint32_t parity) {
  for (int i = 0; i < kSpinLimit; ++i) if (mbar_test_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ bool spin_flag(volatile int* f, int want) {
  for (int i = 0; i < kSpinLimit; ++i) if (*f == want) return true;
  return false;
}

// Thread A (warp 8) signals, thread B (warp 9) answers, `rounds` times.
// TEST 0: A arrives on an mbarrier, both wait with try_wait;  1: A issues 8 MMAs 128x128x16 and a
// tcgen05.commit instead of the arrive;  2: both spin on test_wait;  3: plain volatile flags.
// BG 1: warps 0-7 run ex2 and TMEM load / store in a loop until A is done.  Every wait is bounded.
template <int TEST, int BG>
__global__ void __launch_bounds__(384, 1) probe_handover(long long* out, int rounds) {
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* base = (unsigned char*)(((uintptr_t)smem + 1023) & ~(uintptr_t)1023);
  __shared__ uint64_t bar1, bar2;
  __shared__ uint32_t tmem_base_s;
  __shared__ volatile int done, abort_flag, flag1, flag2;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  for (int i = threadIdx.x; i < 64 * 1024 / 4; i += 384) ((uint32_t*)base)[i] = 0x3c003c00u;
  if (threadIdx.x == 0) {
    done = 0; abort_flag = 0; flag1 = 0; flag2 = 0;
    mbar_init(&bar1, 1); mbar_init(&bar2, 1);
    fence_mbar_init();
  }
  fence_proxy_async_smem();
  if (warp == 0) { tmem_alloc(&tmem_base_s, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  const long long limit = 100000000LL;
  if (warp < 8) {
    if (BG) {
      float x = 0.001f * threadIdx.x, acc = 0.f;
      uint32_t r[32];
      const uint32_t t_s = tmem + ((uint32_t)((warp % 4) * 32) << 16) + 256 + (warp / 4) * 64;
      for (int spin = 0; spin < kSpinLimit && !done; ++spin) {
#pragma unroll
        for (int i = 0; i < 32; ++i) { acc += ex2(x - i); x = fmaf(x, 0.999f, 0.0001f); }
        tmem_ld_32x32b_x32(t_s, r);
        tmem_ld_wait();
        r[0] += __float_as_uint(acc);
        tmem_st_32x32b_x32(t_s + 32, r);
        tmem_st_wait();
      }
      if (acc == 12345.f) out[blockIdx.x * 4 + 3] = 1;
    }
  } else if (warp == 8) {
    const bool leader = elect_one();
    const uint32_t a_addr = smem_addr(base), b_addr = smem_addr(base + 32768);
    const uint32_t id_qk = make_idesc_bf16(128, 128, false, false);
    uint64_t da[8], db[8];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      const uint32_t off = (ks / 4) * 16384 + (ks % 4) * 32;
      da[ks] = make_smem_desc_sw128(a_addr + off, 16, 1024);
      db[ks] = make_smem_desc_sw128(b_addr + off, 16, 1024);
    }
    const long long t0 = clock64();
    bool ok = true;
    for (int r = 0; r < rounds && ok; ++r) {
      if (TEST == 3) {
        if (leader) flag1 = r + 1;
        ok = spin_flag(&flag2, r + 1);
      } else {
        if (TEST == 1) {
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            if (leader) mma_ss(tmem, da[ks], db[ks], id_qk, ks > 0);
          if (leader) mma_commit(&bar1);
        } else if (leader) {
          mbar_arrive(&bar1);
        }
        ok = TEST == 2 ? spin_test(&bar2, r & 1) : mbar_wait(&bar2, r & 1, (volatile int*)&abort_flag, limit);
      }
    }
    const long long t1 = clock64();
    if (leader) { out[blockIdx.x * 4 + 0] = t1 - t0; out[blockIdx.x * 4 + 1] = ok; }
    __syncwarp();
    done = 1;
  } else if (warp == 9 && lane == 0) {
    bool ok = true;
    for (int r = 0; r < rounds && ok; ++r) {
      if (TEST == 3) {
        ok = spin_flag(&flag1, r + 1);
        flag2 = r + 1;
      } else {
        ok = TEST == 2 ? spin_test(&bar1, r & 1) : mbar_wait(&bar1, r & 1, (volatile int*)&abort_flag, limit);
        mbar_arrive(&bar2);
      }
    }
    if (!ok) abort_flag = 1;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

template <int TEST, int BG>
int launch_handover(long long* out, int rounds, int grid) {
  const size_t smem = 64 * 1024 + 1024;
  if (cudaFuncSetAttribute(probe_handover<TEST, BG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return -1;
  probe_handover<TEST, BG><<<grid, 384, smem>>>(out, rounds);
  const cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) { printf("cuda error %s\n", cudaGetErrorString(e)); return -2; }
  return 0;
}

}  // namespace

// out: int64[4 * grid] = per CTA {cycles of all rounds, 1 if no wait gave up, -, -}
extern "C" int run_probe_handover(long long* out, int test, int busy, int rounds, int grid) {
#define HANDOVER_CASE(T, B) if (test == T && busy == B) return launch_handover<T, B>(out, rounds, grid);
  HANDOVER_CASE(0, 0) HANDOVER_CASE(1, 0) HANDOVER_CASE(2, 0) HANDOVER_CASE(3, 0)
  HANDOVER_CASE(0, 1) HANDOVER_CASE(1, 1) HANDOVER_CASE(2, 1) HANDOVER_CASE(3, 1)
#undef HANDOVER_CASE
  return -3;
}
