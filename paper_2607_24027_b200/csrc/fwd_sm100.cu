// Sol-Attn fused forward (Algorithm 1) for sm_100a: TMA + tcgen05.mma + TMEM.
//
// Persistent kernel, two CTAs per SM, d = 128, block_q = block_k = 128.  A CTA owns one query
// block at a time and is split into warp roles that talk through mbarriers:
//
//   router   (warp 4)  pulls (head, query block) work items from a global counter and walks the
//                      pooled keys in chunks of 128 blocks.  For every block it evaluates the
//                      proxy s_ij = scale * Qbar_i . KC_j (Eq. 3) in fp32 and compares it with
//                      tau_i (Eq. 4).  The decision only ever lives in a small shared-memory
//                      record (selected list + per-column bias); nothing of the proxy map goes
//                      to global memory.
//   producer (warp 5)  reads the records and issues TMA loads: one approximate tile per chunk
//                      (KC chunk, mean-V chunk) and K_j / V_j ONLY for routed blocks.
//   mma      (warp 6)  one thread issues tcgen05.mma: S = Q K^T into TMEM, then O += P V with P
//                      read from TMEM (where the softmax warps left it) and V from shared memory.
//   softmax  (warps 0-3, one thread per query row) online softmax over the tile stream; both
//                      branches update the same (m, l, O): an approximate tile is an ordinary
//                      tile whose columns carry the bias log2(n_j) (Eqs. 9-10: multiplicity n_j
//                      in the denominator, mean value times n_j in the numerator) or -inf for
//                      routed / padded columns.  O is rescaled lazily, only when the running
//                      maximum grows by more than 2^8.
//
// Every mbarrier wait is bounded: when one expires the CTA records SOL_ERR_DEVICE_TIMEOUT in the
// workspace status word, all roles drain, TMEM is released and the kernel returns.
#include "common.cuh"
#include "ptx_sm100.cuh"
#include "tmap.cuh"

namespace sol {
namespace {

using namespace ptx;

constexpr int kD = 128;
constexpr int kBlk = 128;
constexpr int kThreads = 256;
constexpr int kTileBytes = kBlk * kD * 2;       // 32 KB: one K-like or V-like tile
constexpr int kHalfBytes = kTileBytes / 2;      // 16 KB: 64 channels x 128 rows (one TMA box)
constexpr int kStages = 2;                      // ring of K/V tiles
constexpr int kRecords = 4;                     // ring of routing records
constexpr int kTmemCols = 256;                  // S: [0,128)  O: [128,256);  P (bf16) aliases S [0,64)
constexpr float kRescaleThreshold = 8.0f;       // log2 units

constexpr uint8_t kRecFirst = 1, kRecLast = 2, kRecApprox = 4;

struct Record {
  int32_t work;                 // bh * Nq + i, or -1: no more work
  int16_t chunk;
  uint8_t flags;
  uint8_t n_sel;
  uint8_t sel[kBlk];            // offsets (within the chunk) of the routed blocks
  float bias[kBlk];             // approximate-tile column bias: log2(n_j), or -inf
};

struct Shared {
  Record rec[kRecords];
  uint64_t rec_full[kRecords], rec_empty[kRecords];
  uint64_t kv_full[kStages], kv_empty[kStages];
  uint64_t q_full, q_empty;
  uint64_t s_full, p_full, pv_done;
  uint32_t tmem_base;
  int abort_flag;
};

struct Params {
  const float* qbar;            // [BH][Nq][d]
  const float* kc;              // [BH][Nk][d]
  const float* tau;             // [BH][Nq]
  __nv_bfloat16* out;
  int32_t* counts;
  uint32_t* mask_out;
  int32_t* status;              // workspace status words
  int N, Nq, Nk, total_work, mode;
  float scale;
};

__device__ __forceinline__ void flag_abort(Shared& sm, const Params& p, int where) {
  sm.abort_flag = 1;
  atomicExch(p.status + kStatusDevice, (int)SOL_ERR_DEVICE_TIMEOUT);
  atomicExch(p.status + kStatusDetail, where);
}

#define SOL_WAIT(bar, parity, where)                                  \
  if (!mbar_wait((bar), (parity), &sm.abort_flag)) {                  \
    flag_abort(sm, p, (where));                                       \
    break;                                                            \
  }

// ------------------------------------------------------------------------------------------------
// router: one warp
__device__ void router_role(Shared& sm, const Params& p, int lane) {
  const unsigned full = 0xffffffffu;
  uint32_t n_rec = 0;
  const int n_chunks = ceil_div(p.Nk, kBlk);
  const int mask_words = ceil_div(p.Nk, 32);
  bool alive = true;
  while (alive) {
    int w = 0;
    if (lane == 0) w = atomicAdd(p.status + kStatusTileCounter, 1);
    w = __shfl_sync(full, w, 0);
    if (w >= p.total_work) break;
    const int bh = w / p.Nq, i = w - bh * p.Nq;
    float4 qb = make_float4(0.f, 0.f, 0.f, 0.f);
    float tau_i = 0.f;
    if (p.mode != SOL_MODE_DENSE) {
      qb = *reinterpret_cast<const float4*>(p.qbar + ((size_t)bh * p.Nq + i) * kD + lane * 4);
      tau_i = p.tau[(size_t)bh * p.Nq + i];
    }
    const float* kc_head = p.kc + (size_t)bh * p.Nk * kD;
    int count = 0;
    for (int t = 0; t < n_chunks; ++t) {
      Record& rec = sm.rec[n_rec % kRecords];
      if (!mbar_wait(&sm.rec_empty[n_rec % kRecords], ((n_rec / kRecords) & 1) ^ 1, &sm.abort_flag)) {
        if (lane == 0) flag_abort(sm, p, 100);
        alive = false;
        break;
      }
      const int j0 = t * kBlk;
      int n_sel = 0;
      bool any_unselected = false;
#pragma unroll 1
      for (int g = 0; g < kBlk / 32; ++g) {
        const int jbase = j0 + g * 32;
        bool sel;
        const int j = jbase + lane;
        if (p.mode == SOL_MODE_DENSE) {
          sel = j < p.Nk;
        } else {
          // partial dot products of 32 pooled keys (lane owns channels 4*lane..4*lane+3), then a
          // transposing butterfly leaves the full dot product of key jbase+l in lane l
          float v[32];
#pragma unroll
          for (int r = 0; r < 32; ++r) {
            const int jr = min(jbase + r, p.Nk - 1);
            const float4 kk = __ldg(reinterpret_cast<const float4*>(kc_head + (size_t)jr * kD + lane * 4));
            v[r] = fmaf(qb.x, kk.x, fmaf(qb.y, kk.y, fmaf(qb.z, kk.z, qb.w * kk.w)));
          }
#pragma unroll
          for (int off = 16; off >= 1; off >>= 1) {
#pragma unroll
            for (int r = 0; r < off; ++r) {
              const bool up = (lane & off) != 0;
              const float send = up ? v[r] : v[r + off];
              const float keep = up ? v[r + off] : v[r];
              v[r] = keep + __shfl_xor_sync(full, send, off);
            }
          }
          sel = (j < p.Nk) && (p.scale * v[0] > tau_i);
        }
        const unsigned m = __ballot_sync(full, sel);
        const bool valid = j < p.Nk;
        any_unselected |= (valid && !sel);
        rec.bias[g * 32 + lane] = (valid && !sel) ? log2f((float)min(kBlk, p.N - j * kBlk)) : -INFINITY;
        if (sel) rec.sel[n_sel + __popc(m & ((1u << lane) - 1u))] = (uint8_t)(g * 32 + lane);
        n_sel += __popc(m);
        if (p.mask_out && lane == 0 && jbase < p.Nk) p.mask_out[(size_t)w * mask_words + jbase / 32] = m;
      }
      any_unselected = __any_sync(full, any_unselected);
      count += n_sel;
      if (lane == 0) {
        rec.work = w;
        rec.chunk = (int16_t)t;
        rec.n_sel = (uint8_t)n_sel;     // n_sel <= 128 fits
        rec.flags = (t == 0 ? kRecFirst : 0) | (t == n_chunks - 1 ? kRecLast : 0) |
                    ((p.mode == SOL_MODE_SOL && any_unselected) ? kRecApprox : 0);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.rec_full[n_rec % kRecords]);
      ++n_rec;
    }
    if (alive && lane == 0 && p.counts) p.counts[w] = count;
  }
  // end-of-stream record
  if (alive) {
    if (mbar_wait(&sm.rec_empty[n_rec % kRecords], ((n_rec / kRecords) & 1) ^ 1, &sm.abort_flag)) {
      if (lane == 0) {
        sm.rec[n_rec % kRecords].work = -1;
        mbar_arrive(&sm.rec_full[n_rec % kRecords]);
      }
    } else if (lane == 0) {
      flag_abort(sm, p, 101);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// producer: one thread
__device__ void producer_role(Shared& sm, const Params& p, unsigned char* sQ, unsigned char* sKV,
                              const CUtensorMap* tm_q, const CUtensorMap* tm_k, const CUtensorMap* tm_v,
                              const CUtensorMap* tm_kc, const CUtensorMap* tm_vm) {
  uint32_t n_rec = 0, n_load = 0, n_item = 0;
  auto load_tile = [&](const CUtensorMap* tm, int row, int bh) -> bool {
    const uint32_t s = n_load % kStages;
    if (!mbar_wait(&sm.kv_empty[s], ((n_load / kStages) & 1) ^ 1, &sm.abort_flag)) return false;
    mbar_arrive_expect_tx(&sm.kv_full[s], kTileBytes);
    unsigned char* dst = sKV + (size_t)s * kTileBytes;
    tma_load_3d(dst, tm, &sm.kv_full[s], 0, row, bh);
    tma_load_3d(dst + kHalfBytes, tm, &sm.kv_full[s], 64, row, bh);
    ++n_load;
    return true;
  };
  for (;;) {
    const uint32_t r = n_rec % kRecords;
    SOL_WAIT(&sm.rec_full[r], (n_rec / kRecords) & 1, 200);
    const Record& rec = sm.rec[r];
    const int w = rec.work;
    if (w < 0) break;
    const int bh = w / p.Nq, i = w - bh * p.Nq;
    const int j0 = rec.chunk * kBlk;
    bool ok = true;
    if (rec.flags & kRecFirst) {
      SOL_WAIT(&sm.q_empty, (n_item & 1) ^ 1, 201);
      mbar_arrive_expect_tx(&sm.q_full, kTileBytes);
      tma_load_3d(sQ, tm_q, &sm.q_full, 0, i * kBlk, bh);
      tma_load_3d(sQ + kHalfBytes, tm_q, &sm.q_full, 64, i * kBlk, bh);
      ++n_item;
    }
    if (rec.flags & kRecApprox) ok = load_tile(tm_kc, j0, bh) && load_tile(tm_vm, j0, bh);
    const int n_sel = rec.n_sel;
    for (int e = 0; ok && e < n_sel; ++e) {
      const int row = (j0 + rec.sel[e]) * kBlk;
      ok = load_tile(tm_k, row, bh) && load_tile(tm_v, row, bh);
    }
    if (!ok) { flag_abort(sm, p, 202); break; }
    mbar_arrive(&sm.rec_empty[r]);
    ++n_rec;
  }
  if (sm.abort_flag) {
    // let copies that are still in flight land before the CTA's shared memory goes away
    int never = 0;                                   // this drain must not be cut short by the abort flag
    for (uint32_t back = 0; back < kStages && back < n_load; ++back) {
      const uint32_t n = n_load - 1 - back;
      mbar_wait(&sm.kv_full[n % kStages], (n / kStages) & 1, &never);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// mma issuer: one thread
__device__ void mma_role(Shared& sm, const Params& p, unsigned char* sQ, unsigned char* sKV, uint32_t tmem) {
  const uint32_t idesc_qk = make_idesc_bf16(kBlk, kBlk, false, false);
  const uint32_t idesc_pv = make_idesc_bf16(kBlk, kD, false, true);
  const uint32_t q_addr = smem_addr(sQ), kv_addr = smem_addr(sKV);
  const uint32_t tmem_s = tmem, tmem_o = tmem + 128;
  uint32_t n_rec = 0, n_load = 0, n_item = 0, g = 0;   // g: tiles issued so far by this CTA
  int tiles_in_item = 0;
  for (;;) {
    const uint32_t r = n_rec % kRecords;
    SOL_WAIT(&sm.rec_full[r], (n_rec / kRecords) & 1, 300);
    const Record& rec = sm.rec[r];
    if (rec.work < 0) break;
    const uint8_t flags = rec.flags;
    const int n_tiles = ((flags & kRecApprox) ? 1 : 0) + rec.n_sel;
    mbar_arrive(&sm.rec_empty[r]);       // nothing else of the record is needed here
    ++n_rec;
    bool ok = true;
    if (flags & kRecFirst) {
      if (!mbar_wait(&sm.q_full, n_item & 1, &sm.abort_flag)) { flag_abort(sm, p, 301); break; }
      ++n_item;
      tiles_in_item = 0;
    }
    for (int e = 0; e < n_tiles; ++e) {
      // ---- S = Q K^T
      const uint32_t sk = n_load % kStages;
      if (!mbar_wait(&sm.kv_full[sk], (n_load / kStages) & 1, &sm.abort_flag)) { ok = false; break; }
      ++n_load;
      if (g > 0 && !mbar_wait(&sm.pv_done, (g - 1) & 1, &sm.abort_flag)) { ok = false; break; }   // P of the previous tile consumed
      tc_fence_after();
#pragma unroll
      for (int ks = 0; ks < kD / 16; ++ks) {
        const uint32_t off = (ks / 4) * kHalfBytes + (ks % 4) * 32;
        mma_ss(tmem_s, make_smem_desc_sw128(q_addr + off, 16, 1024),
               make_smem_desc_sw128(kv_addr + sk * kTileBytes + off, 16, 1024), idesc_qk, ks > 0);
      }
      mma_commit(&sm.kv_empty[sk]);
      mma_commit(&sm.s_full);
      // ---- O += P V
      const uint32_t sv = n_load % kStages;
      if (!mbar_wait(&sm.kv_full[sv], (n_load / kStages) & 1, &sm.abort_flag)) { ok = false; break; }
      ++n_load;
      if (!mbar_wait(&sm.p_full, g & 1, &sm.abort_flag)) { ok = false; break; }
      tc_fence_after();
#pragma unroll
      for (int ks = 0; ks < kBlk / 16; ++ks) {
        mma_ts(tmem_o, tmem_s + ks * 8, make_smem_desc_sw128(kv_addr + sv * kTileBytes + ks * 2048, kHalfBytes, 1024),
               idesc_pv, (tiles_in_item > 0 || ks > 0) ? 1u : 0u);
      }
      mma_commit(&sm.kv_empty[sv]);
      mma_commit(&sm.pv_done);
      ++g;
      ++tiles_in_item;
    }
    if (!ok) { flag_abort(sm, p, 302); break; }
    if (flags & kRecLast) mma_commit(&sm.q_empty);     // every MMA that reads Q_i has been issued
  }
}

// ------------------------------------------------------------------------------------------------
// softmax + correction + epilogue: 128 threads, thread = query row
__device__ void softmax_role(Shared& sm, const Params& p, uint32_t tmem, int warp, int lane) {
  const unsigned full = 0xffffffffu;
  const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
  const uint32_t t_s = lane_base, t_o = lane_base + 128;
  const int row = warp * 32 + lane;
  const float sl2 = p.scale * 1.4426950408889634f;
  uint32_t n_rec = 0, g = 0;
  int tiles_in_item = 0;
  float m_used = 0.f, l = 0.f;
  bool alive = true;
  while (alive) {
    const uint32_t r = n_rec % kRecords;
    if (!mbar_wait(&sm.rec_full[r], (n_rec / kRecords) & 1, &sm.abort_flag)) { flag_abort(sm, p, 400); break; }
    const Record& rec = sm.rec[r];
    const int w = rec.work;
    if (w < 0) break;
    const uint8_t flags = rec.flags;
    const int n_sel = rec.n_sel;
    const int n_tiles = ((flags & kRecApprox) ? 1 : 0) + n_sel;
    const int j0 = rec.chunk * kBlk;
    if (flags & kRecFirst) tiles_in_item = 0;
    for (int e = 0; e < n_tiles; ++e) {
      const bool approx = (flags & kRecApprox) && e == 0;
      int cols_valid = kBlk;
      if (!approx) {
        const int j = j0 + rec.sel[e - ((flags & kRecApprox) ? 1 : 0)];
        cols_valid = min(kBlk, p.N - j * kBlk);
      }
      const bool general = approx || cols_valid < kBlk;
      if (!mbar_wait(&sm.s_full, g & 1, &sm.abort_flag)) { flag_abort(sm, p, 401); alive = false; break; }
      tc_fence_after();
      // ---- pass 1: row maximum (log2 domain)
      float mx = -INFINITY;
#pragma unroll 1
      for (int h = 0; h < 2; ++h) {
        uint32_t a[32], b[32];
        tmem_ld_32x32b_x32(t_s + h * 64, a);
        tmem_ld_32x32b_x32(t_s + h * 64 + 32, b);
        tmem_ld_wait();
        if (!general) {
#pragma unroll
          for (int c = 0; c < 32; ++c) mx = fmaxf(mx, fmaxf(__uint_as_float(a[c]), __uint_as_float(b[c])));
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            const int c0 = h * 64 + c, c1 = c0 + 32;
            const float b0 = approx ? rec.bias[c0] : (c0 < cols_valid ? 0.f : -INFINITY);
            const float b1 = approx ? rec.bias[c1] : (c1 < cols_valid ? 0.f : -INFINITY);
            mx = fmaxf(mx, fmaxf(fmaf(__uint_as_float(a[c]), sl2, b0), fmaf(__uint_as_float(b[c]), sl2, b1)));
          }
        }
      }
      if (!general) mx *= sl2;
      // ---- running maximum, lazy rescale of O
      if (tiles_in_item == 0) {
        m_used = mx;
        l = 0.f;
      } else if (__any_sync(full, mx > m_used + kRescaleThreshold)) {
        const float m_new = fmaxf(m_used, mx);
        const float f = ex2(m_used - m_new);
        if (!mbar_wait(&sm.pv_done, (g - 1) & 1, &sm.abort_flag)) { flag_abort(sm, p, 402); alive = false; break; }
        tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t o[32];
          tmem_ld_32x32b_x32(t_o + c * 32, o);
          tmem_ld_wait();
#pragma unroll
          for (int x = 0; x < 32; ++x) o[x] = __float_as_uint(__uint_as_float(o[x]) * f);
          tmem_st_32x32b_x32(t_o + c * 32, o);
        }
        l *= f;
        m_used = m_new;
      }
      // ---- pass 2: P = exp2(S - m), row sum, P (bf16) back to TMEM over S
#pragma unroll 1
      for (int h = 0; h < 2; ++h) {
        uint32_t a[32], b[32];
        tmem_ld_32x32b_x32(t_s + h * 64, a);
        tmem_ld_32x32b_x32(t_s + h * 64 + 32, b);
        tmem_ld_wait();
        float sum0 = 0.f, sum1 = 0.f;
        if (!general) {
          const float nm = -m_used;
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            const float pa = ex2(fmaf(__uint_as_float(a[c]), sl2, nm));
            const float pb = ex2(fmaf(__uint_as_float(b[c]), sl2, nm));
            sum0 += pa; sum1 += pb;
            a[c] = __float_as_uint(pa); b[c] = __float_as_uint(pb);
          }
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            const int c0 = h * 64 + c, c1 = c0 + 32;
            const float b0 = approx ? rec.bias[c0] : (c0 < cols_valid ? 0.f : -INFINITY);
            const float b1 = approx ? rec.bias[c1] : (c1 < cols_valid ? 0.f : -INFINITY);
            const float pa = ex2(fmaf(__uint_as_float(a[c]), sl2, b0 - m_used));
            const float pb = ex2(fmaf(__uint_as_float(b[c]), sl2, b1 - m_used));
            sum0 += pa; sum1 += pb;
            a[c] = __float_as_uint(pa); b[c] = __float_as_uint(pb);
          }
        }
        l += sum0 + sum1;
        uint32_t pk[32];
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          __nv_bfloat162 x = __floats2bfloat162_rn(__uint_as_float(a[2 * c]), __uint_as_float(a[2 * c + 1]));
          __nv_bfloat162 y = __floats2bfloat162_rn(__uint_as_float(b[2 * c]), __uint_as_float(b[2 * c + 1]));
          pk[c] = *reinterpret_cast<uint32_t*>(&x);
          pk[16 + c] = *reinterpret_cast<uint32_t*>(&y);
        }
        tmem_st_32x32b_x32(t_s + h * 32, pk);
      }
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(&sm.p_full);
      ++g;
      ++tiles_in_item;
    }
    if (!alive) break;
    // ---- end of the work item: O_i = acc / l
    if (flags & kRecLast) {
      const int bh = w / p.Nq, i = w - bh * p.Nq;
      const int q_rows = min(kBlk, p.N - i * kBlk);
      __nv_bfloat16* orow = p.out + ((size_t)bh * p.N + (size_t)i * kBlk + row) * kD;
      if (tiles_in_item > 0) {
        if (!mbar_wait(&sm.pv_done, (g - 1) & 1, &sm.abort_flag)) { flag_abort(sm, p, 403); break; }
        tc_fence_after();
        const float inv = 1.f / l;
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t o[32];
          tmem_ld_32x32b_x32(t_o + c * 32, o);
          tmem_ld_wait();
          if (row < q_rows) {
#pragma unroll
            for (int x = 0; x < 4; ++x) {
              uint4 pk;
              uint32_t* pw = reinterpret_cast<uint32_t*>(&pk);
#pragma unroll
              for (int y = 0; y < 4; ++y) {
                __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(o[x * 8 + 2 * y]) * inv,
                                                          __uint_as_float(o[x * 8 + 2 * y + 1]) * inv);
                pw[y] = *reinterpret_cast<uint32_t*>(&hh);
              }
              *reinterpret_cast<uint4*>(orow + c * 32 + x * 8) = pk;
            }
          }
        }
        tc_fence_before();
      } else if (row < q_rows) {
        // a query block that routed nothing in keep-or-drop mode has no attention mass at all
        for (int c = 0; c < kD; c += 8) *reinterpret_cast<uint4*>(orow + c) = make_uint4(0, 0, 0, 0);
      }
      tiles_in_item = 0;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.rec_empty[r]);
    ++n_rec;
  }
}

__global__ void __launch_bounds__(kThreads, 2)
fwd_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_kc,
                 const __grid_constant__ CUtensorMap tm_vm, const Params p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* sQ = base;
  unsigned char* sKV = base + kTileBytes;
  Shared& sm = *reinterpret_cast<Shared*>(base + kTileBytes + kStages * kTileBytes);
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;

  if (threadIdx.x == 0) {
    sm.abort_flag = 0;
    for (int r = 0; r < kRecords; ++r) { mbar_init(&sm.rec_full[r], 1); mbar_init(&sm.rec_empty[r], 6); }
    for (int s = 0; s < kStages; ++s) { mbar_init(&sm.kv_full[s], 1); mbar_init(&sm.kv_empty[s], 1); }
    mbar_init(&sm.q_full, 1); mbar_init(&sm.q_empty, 1);
    mbar_init(&sm.s_full, 1); mbar_init(&sm.p_full, 128); mbar_init(&sm.pv_done, 1);
    fence_mbar_init();
  }
  if (warp == 5 && lane == 0) {
    prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v);
    prefetch_tensormap(&tm_kc); prefetch_tensormap(&tm_vm);
  }
  if (warp == 0) { tmem_alloc(&sm.tmem_base, kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp < 4) {
    softmax_role(sm, p, tmem, warp, lane);
  } else if (warp == 4) {
    router_role(sm, p, lane);
  } else if (warp == 5) {
    if (lane == 0) producer_role(sm, p, sQ, sKV, &tm_q, &tm_k, &tm_v, &tm_kc, &tm_vm);
  } else if (warp == 6) {
    if (lane == 0) mma_role(sm, p, sQ, sKV, tmem);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace

bool fwd_sm100_supports(const Problem& p) { return p.d == kD && p.block_q == kBlk && p.block_k == kBlk; }

cudaError_t launch_fwd_sm100(const Problem& p, const __nv_bfloat16* q, const __nv_bfloat16* k,
                             const __nv_bfloat16* v, __nv_bfloat16* out, const WsPtrs& ws, const float* tau,
                             int32_t* counts, uint32_t* mask_out, cudaStream_t stream, int* n_launches) {
  CUtensorMap tq, tk, tv, tkc, tvm;
  if (!make_tmap_bf16_3d(&tq, q, p.BH, p.N, kD, kBlk) || !make_tmap_bf16_3d(&tk, k, p.BH, p.N, kD, kBlk) ||
      !make_tmap_bf16_3d(&tv, v, p.BH, p.N, kD, kBlk) || !make_tmap_bf16_3d(&tkc, ws.kcb, p.BH, p.Nk, kD, kBlk) ||
      !make_tmap_bf16_3d(&tvm, ws.vmb, p.BH, p.Nk, kD, kBlk))
    return cudaErrorInvalidValue;
  Params prm{};
  prm.qbar = ws.qbar; prm.kc = ws.kc; prm.tau = tau; prm.out = out; prm.counts = counts; prm.mask_out = mask_out;
  prm.status = ws.status; prm.N = p.N; prm.Nq = p.Nq; prm.Nk = p.Nk; prm.total_work = p.BH * p.Nq;
  prm.mode = p.mode; prm.scale = p.scale;

  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  const size_t smem = 1024 + kTileBytes + kStages * kTileBytes + sizeof(Shared);
  e = cudaFuncSetAttribute(fwd_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int grid = prm.total_work < 2 * sms ? prm.total_work : 2 * sms;
  fwd_sm100_kernel<<<grid, kThreads, smem, stream>>>(tq, tk, tv, tkc, tvm, prm);
  if (n_launches) *n_launches += 1;
  return cudaGetLastError();
}

}  // namespace sol
