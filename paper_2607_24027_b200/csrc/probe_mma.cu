// Microbenchmark behind the tensor-side roofline of the fused kernel: how long one attention tile's
// worth of tcgen05 MMAs takes on an otherwise idle SM (timing only; operands are whatever shared
// memory and TMEM hold), with and without a concurrent stream of bulk copies landing one K and one V
// tile (64 KB) per iteration in shared memory.
//
// Per iteration: 8 score MMAs 128x128x16 (operands: shared x shared, or TMEM x shared) into one of
// two accumulators, then 8 value MMAs 128x128x16 (TMEM x shared, MN-major B) into two others.
// Built and run by `python -m paper_2607_24027_b200.mma_probe`; not part of libsol_attn.so.
#include <cstdio>

#include <cuda_bf16.h>

#include "ptx_sm100.cuh"

using namespace sol::ptx;

// MODE bit 0: copy stream on; bit 1: score MMAs take A from TMEM; bit 2: no MMAs at all;
// bit 3: score MMAs TMEM x shared in two halves of 64 key columns.
// The issuing thread's own instructions must not be what is measured: the mode is a template
// parameter and every descriptor is built before the timed loop.
template <int MODE>
__global__ void __launch_bounds__(128) probe_mma(long long* out, const unsigned char* gsrc, int iters, int src_bytes) {
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* base = (unsigned char*)(((uintptr_t)smem + 1023) & ~(uintptr_t)1023);
  __shared__ uint64_t bar, tbar[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  const int warp = threadIdx.x / 32;
  for (int i = threadIdx.x; i < 160 * 1024 / 4; i += 128) ((uint32_t*)base)[i] = 0x3c003c00u;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(&bar, 1); mbar_init(&tbar[0], 1); mbar_init(&tbar[1], 1);
    fence_mbar_init();
  }
  fence_proxy_async_smem();
  if (warp == 0) { tmem_alloc(&tmem_base_s, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  const unsigned char* src = gsrc + (size_t)blockIdx.x * src_bytes;
  if (threadIdx.x == 0 && !(MODE & 4)) {
    const uint32_t a_addr = smem_addr(base), b_addr = smem_addr(base + 32768);
    const uint32_t id_qk = make_idesc_bf16(128, 128, false, false);
    const uint32_t id_qk64 = make_idesc_bf16(128, 64, false, false);
    const uint32_t id_pv = make_idesc_bf16(128, 128, false, true);
    uint64_t da[8], db[8], db2[8], dv[8];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      const uint32_t off = (ks / 4) * 16384 + (ks % 4) * 32;
      da[ks] = make_smem_desc_sw128(a_addr + off, 16, 1024);
      db[ks] = make_smem_desc_sw128(b_addr + off, 16, 1024);
      db2[ks] = make_smem_desc_sw128(b_addr + off + 8192, 16, 1024);
      dv[ks] = make_smem_desc_sw128(b_addr + 32768 + ks * 2048, 16384, 1024);
    }
    const long long t0 = clock64();
#pragma unroll 1
    for (int it = 0; it < iters; it += 2) {
#pragma unroll
      for (int u = 0; u < 2; ++u) {               // two tiles per trip: the accumulator choice is static
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          if (MODE & 8) {
            mma_ts(tmem + u * 128, tmem + 256 + ks * 8, db[ks], id_qk64, ks > 0);
            mma_ts(tmem + u * 128 + 64, tmem + 256 + ks * 8, db2[ks], id_qk64, ks > 0);
          } else if (MODE & 2) {
            mma_ts(tmem + u * 128, tmem + 256 + ks * 8, db[ks], id_qk, ks > 0);
          } else {
            mma_ss(tmem + u * 128, da[ks], db[ks], id_qk, ks > 0);
          }
        }
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) mma_ts(tmem + 256 + (ks / 4) * 128, tmem + (1 - u) * 128 + ks * 8, dv[ks], id_pv, 1);
      }
    }
    const long long t1 = clock64();
    mma_commit(&bar);
    const bool ok = mbar_wait(&bar, 0, &abort_flag);
    out[blockIdx.x * 4 + 0] = clock64() - t0;
    out[blockIdx.x * 4 + 2] = ok ? (t1 - t0) : -1;      // issue time alone (the loop), or -1 on a timeout
  }
  if (threadIdx.x == 32 && (MODE & 1)) {
    const long long t0 = clock64();
    bool ok = true;
    for (int it = 0; it < iters && ok; ++it) {
      for (int half = 0; half < 2; ++half) {
        const int n = it * 2 + half;
        if (n >= 2) ok = ok && mbar_wait(&tbar[n & 1], ((n - 2) >> 1) & 1, &abort_flag);
        mbar_arrive_expect_tx(&tbar[n & 1], 32768);
        bulk_load_1d(base + 96 * 1024 + (n & 1) * 32768, src + ((size_t)n * 32768) % src_bytes, 32768, &tbar[n & 1]);
      }
    }
    const int last = iters * 2 - 1;
    ok = ok && mbar_wait(&tbar[last & 1], (last >> 1) & 1, &abort_flag);
    ok = ok && mbar_wait(&tbar[(last - 1) & 1], ((last - 1) >> 1) & 1, &abort_flag);
    out[blockIdx.x * 4 + 1] = clock64() - t0;
    out[blockIdx.x * 4 + 3] = ok;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

template <int MODE>
static int launch(long long* out_dev, const unsigned char* src, int iters, int grid, int src_bytes) {
  const size_t smem = 160 * 1024 + 1024;
  if (cudaFuncSetAttribute(probe_mma<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return -1;
  probe_mma<MODE><<<grid, 128, smem>>>(out_dev, src, iters, src_bytes);
  const cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) { printf("cuda error %s\n", cudaGetErrorString(e)); return -2; }
  return 0;
}

// out_dev: int64[4 * grid] = per CTA {MMA cycles, copy cycles, MMA issue cycles, copy ok}; src: grid * src_bytes bytes;
// iters must be even
extern "C" int run_probe_mma(long long* out_dev, const unsigned char* src, int mode, int iters, int grid, int src_bytes) {
  switch (mode) {
    case 0: return launch<0>(out_dev, src, iters, grid, src_bytes);
    case 1: return launch<1>(out_dev, src, iters, grid, src_bytes);
    case 2: return launch<2>(out_dev, src, iters, grid, src_bytes);
    case 3: return launch<3>(out_dev, src, iters, grid, src_bytes);
    case 5: return launch<5>(out_dev, src, iters, grid, src_bytes);
    case 8: return launch<8>(out_dev, src, iters, grid, src_bytes);
    case 9: return launch<9>(out_dev, src, iters, grid, src_bytes);
    default: return -3;
  }
}
