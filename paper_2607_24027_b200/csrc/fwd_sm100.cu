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
constexpr int kPolyEvery = 4;                   // every 4th exp2 runs on the FMA pipe (0: none)
constexpr int kSoftmaxRegs = 184, kOtherRegs = 72;   // setmaxnreg split of the 2 x 128 x 128 budget

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

// 2^x for x <= ~8 without the MUFU unit: round-to-nearest split x = n + f, f in [-0.5, 0.5],
// cubic minimax polynomial for 2^f (max relative error 7.5e-5, far below bf16 resolution), and n
// added straight into the exponent field.
__device__ __forceinline__ float exp2_poly(float x) {
  x = fmaxf(x, -126.f);
  const float magic = 12582912.f;               // 1.5 * 2^23: the low mantissa bits of x + magic hold n
  const float r = x + magic;
  const float f = x - (r - magic);
  const float pz = fmaf(fmaf(fmaf(0.055171460f, f, 0.24261086f), f, 0.69326097f), f, 0.99992812f);
  return __int_as_float(__float_as_int(pz) + (__float_as_int(r) << 23));
}

// Optional per-role cycle accounting (build with -DSOL_PROFILE): how long each role spends in
// each kind of wait.  Slot meaning is listed next to every use; read back with
// sol_attn_debug_profile().
#ifdef SOL_PROFILE
constexpr int kProfCtas = 512, kProfRoles = 4, kProfSlots = 8;
__device__ long long g_prof[kProfCtas * kProfRoles * kProfSlots];
struct Prof {
  long long v[kProfSlots];
  long long t0;
  __device__ Prof() {
    for (int i = 0; i < kProfSlots; ++i) v[i] = 0;
    t0 = clock64();
  }
  __device__ void flush(int role) {
    v[kProfSlots - 1] = clock64() - t0;
    if (blockIdx.x < kProfCtas)
      for (int i = 0; i < kProfSlots; ++i) g_prof[(blockIdx.x * kProfRoles + role) * kProfSlots + i] = v[i];
  }
};
__device__ __forceinline__ bool prof_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, long long& acc) {
  const long long t = clock64();
  const bool ok = mbar_wait(bar, parity, abort_flag);
  acc += clock64() - t;
  return ok;
}
#define WAIT(bar, parity, slot) prof_wait((bar), (parity), &sm.abort_flag, prof.v[slot])
#define PROF_DECL Prof prof;
#define PROF_COUNT(slot) (++prof.v[slot])
#define PROF_FLUSH(role) prof.flush(role)
#else
#define WAIT(bar, parity, slot) mbar_wait((bar), (parity), &sm.abort_flag)
#define PROF_DECL
#define PROF_COUNT(slot)
#define PROF_FLUSH(role)
#endif

#define SOL_WAIT(bar, parity, where, slot)                            \
  if (!WAIT((bar), (parity), (slot))) {                               \
    flag_abort(sm, p, (where));                                       \
    break;                                                            \
  }

// ------------------------------------------------------------------------------------------------
// router: one warp
__device__ void router_role(Shared& sm, const Params& p, int lane) {
  PROF_DECL
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
      if (!WAIT(&sm.rec_empty[n_rec % kRecords], ((n_rec / kRecords) & 1) ^ 1, 0)) {   // prof 0: record ring full
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
          // lane owns channels 4*lane..4*lane+3.  Eight pooled keys at a time: partial dot
          // products, a transposing butterfly over lane bits 0-2 and two plain exchanges leave the
          // dot product of key (8*sub + (lane & 7)) in every lane; lanes 8*sub..8*sub+7 keep it.
          float dot = 0.f;
#pragma unroll 1
          for (int sub = 0; sub < 4; ++sub) {
            float v[8];
#pragma unroll
            for (int r = 0; r < 8; ++r) {
              const int jr = min(jbase + sub * 8 + r, p.Nk - 1);
              const float4 kk = __ldg(reinterpret_cast<const float4*>(kc_head + (size_t)jr * kD + lane * 4));
              v[r] = fmaf(qb.x, kk.x, fmaf(qb.y, kk.y, fmaf(qb.z, kk.z, qb.w * kk.w)));
            }
#pragma unroll
            for (int off = 4; off >= 1; off >>= 1) {
#pragma unroll
              for (int r = 0; r < off; ++r) {
                const bool up = (lane & off) != 0;
                const float send = up ? v[r] : v[r + off];
                const float keep = up ? v[r + off] : v[r];
                v[r] = keep + __shfl_xor_sync(full, send, off);
              }
            }
            v[0] += __shfl_xor_sync(full, v[0], 8);
            v[0] += __shfl_xor_sync(full, v[0], 16);
            if ((lane >> 3) == sub) dot = v[0];
          }
          sel = (j < p.Nk) && (p.scale * dot > tau_i);
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
  PROF_FLUSH(0);
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
  PROF_DECL
  auto load_tile = [&](const CUtensorMap* tm, int row, int bh) -> bool {
    const uint32_t s = n_load % kStages;
    if (!WAIT(&sm.kv_empty[s], ((n_load / kStages) & 1) ^ 1, 1)) return false;   // prof 1: K/V ring full
    mbar_arrive_expect_tx(&sm.kv_full[s], kTileBytes);
    unsigned char* dst = sKV + (size_t)s * kTileBytes;
    tma_load_3d(dst, tm, &sm.kv_full[s], 0, row, bh);
    tma_load_3d(dst + kHalfBytes, tm, &sm.kv_full[s], 64, row, bh);
    ++n_load;
    return true;
  };
  for (;;) {
    const uint32_t r = n_rec % kRecords;
    SOL_WAIT(&sm.rec_full[r], (n_rec / kRecords) & 1, 200, 0);                   // prof 0: no record yet
    const Record& rec = sm.rec[r];
    const int w = rec.work;
    if (w < 0) break;
    const int bh = w / p.Nq, i = w - bh * p.Nq;
    const int j0 = rec.chunk * kBlk;
    bool ok = true;
    if (rec.flags & kRecFirst) {
      SOL_WAIT(&sm.q_empty, (n_item & 1) ^ 1, 201, 2);                         // prof 2: Q slot busy
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
  PROF_FLUSH(1);
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
  PROF_DECL
  for (;;) {
    const uint32_t r = n_rec % kRecords;
    SOL_WAIT(&sm.rec_full[r], (n_rec / kRecords) & 1, 300, 0);                   // prof 0: no record yet
    const Record& rec = sm.rec[r];
    if (rec.work < 0) break;
    const uint8_t flags = rec.flags;
    const int n_tiles = ((flags & kRecApprox) ? 1 : 0) + rec.n_sel;
    mbar_arrive(&sm.rec_empty[r]);       // nothing else of the record is needed here
    ++n_rec;
    bool ok = true;
    if (flags & kRecFirst) {
      if (!WAIT(&sm.q_full, n_item & 1, 1)) { flag_abort(sm, p, 301); break; }      // prof 1: Q not loaded
      ++n_item;
      tiles_in_item = 0;
    }
    for (int e = 0; e < n_tiles; ++e) {
      // ---- S = Q K^T
      const uint32_t sk = n_load % kStages;
      if (!WAIT(&sm.kv_full[sk], (n_load / kStages) & 1, 2)) { ok = false; break; }   // prof 2: K not loaded
      ++n_load;
      if (g > 0 && !WAIT(&sm.pv_done, (g - 1) & 1, 3)) { ok = false; break; }         // prof 3: previous P V still running
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
      if (!WAIT(&sm.kv_full[sv], (n_load / kStages) & 1, 4)) { ok = false; break; }   // prof 4: V not loaded
      ++n_load;
      if (!WAIT(&sm.p_full, g & 1, 5)) { ok = false; break; }                         // prof 5: softmax not done
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
  PROF_FLUSH(2);
}

// ------------------------------------------------------------------------------------------------
// softmax + correction + epilogue: 128 threads, thread = query row
__device__ void softmax_role(Shared& sm, const Params& p, uint32_t tmem, int warp, int lane) {
  const unsigned full = 0xffffffffu;
  const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
  const uint32_t t_s = lane_base, t_o = lane_base + 128;
  const int row = warp * 32 + lane;
  const float sl2 = p.scale * 1.4426950408889634f;
  const float inv_sl2 = 1.f / sl2;
  uint32_t n_rec = 0, g = 0;
  int tiles_in_item = 0;
  float m_used = 0.f, l = 0.f;
  bool alive = true;
  PROF_DECL
  while (alive) {
    const uint32_t r = n_rec % kRecords;
    if (!WAIT(&sm.rec_full[r], (n_rec / kRecords) & 1, 0)) { flag_abort(sm, p, 400); break; }   // prof 0: no record yet
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
      if (!WAIT(&sm.s_full, g & 1, 1)) { flag_abort(sm, p, 401); alive = false; break; }   // prof 1: S not ready
      tc_fence_after();
      // ---- the whole row of S (128 fp32) into registers with one wait
      uint32_t sr[kBlk];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld_32x32b_x32(t_s + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[c * 32]));
      tmem_ld_wait();
      if (general) {
        // bring the rare tiles (approximate chunk, ragged last block) to the common form
        // logit = sl2 * x by folding the column bias into x; -inf marks masked columns
#pragma unroll
        for (int c = 0; c < kBlk; ++c) {
          const float x = __uint_as_float(sr[c]);
          sr[c] = __float_as_uint(approx ? fmaf(rec.bias[c], inv_sl2, x) : (c < cols_valid ? x : -INFINITY));
        }
      }
      float mx;
      {
        float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          m0 = fmaxf(m0, __uint_as_float(sr[c]));
          m1 = fmaxf(m1, __uint_as_float(sr[32 + c]));
          m2 = fmaxf(m2, __uint_as_float(sr[64 + c]));
          m3 = fmaxf(m3, __uint_as_float(sr[96 + c]));
        }
        mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)) * sl2;
      }
      // ---- running maximum, lazy rescale of O
      if (tiles_in_item == 0) {
        m_used = mx;
        l = 0.f;
      } else if (__any_sync(full, mx > m_used + kRescaleThreshold)) {
        const float m_new = fmaxf(m_used, mx);
        const float f = ex2(m_used - m_new);
        PROF_COUNT(4);                                                                   // prof 4: number of rescales
        if (!WAIT(&sm.pv_done, (g - 1) & 1, 2)) { flag_abort(sm, p, 402); alive = false; break; }
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
      // ---- P = exp2(sl2 * S - m): most elements on the MUFU unit, every kPolyEvery-th one as a
      //      polynomial on the FMA pipe; row sum; P (bf16) back to TMEM over the first half of S
      {
        const float nm = -m_used;
        float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;
#pragma unroll
        for (int c = 0; c < kBlk; c += 4) {
          float e[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float x = fmaf(__uint_as_float(sr[c + u]), sl2, nm);
            e[u] = (kPolyEvery > 0 && ((c + u) % kPolyEvery) == kPolyEvery - 1) ? exp2_poly(x) : ex2(x);
          }
          sum0 += e[0]; sum1 += e[1]; sum2 += e[2]; sum3 += e[3];
          __nv_bfloat162 lo = __floats2bfloat162_rn(e[0], e[1]);
          __nv_bfloat162 hi = __floats2bfloat162_rn(e[2], e[3]);
          sr[c / 2] = *reinterpret_cast<uint32_t*>(&lo);
          sr[c / 2 + 1] = *reinterpret_cast<uint32_t*>(&hi);
        }
        l += (sum0 + sum1) + (sum2 + sum3);
        tmem_st_32x32b_x32(t_s, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
        tmem_st_32x32b_x32(t_s + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
      }
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(&sm.p_full);
      PROF_COUNT(5);                                                                     // prof 5: tiles
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
        if (!WAIT(&sm.pv_done, (g - 1) & 1, 3)) { flag_abort(sm, p, 403); break; }           // prof 3: last P V of the item
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
  if (lane == 0 && warp == 0) PROF_FLUSH(3);
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
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
    softmax_role(sm, p, tmem, warp, lane);
  } else {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));
  }
  if (warp == 4) {
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

#ifdef SOL_PROFILE
}  // namespace sol
// Debug builds only: copies the per-CTA, per-role wait-cycle counters of the last launch to the host.
extern "C" int sol_attn_debug_profile(long long* host_out, int n_values) {
  const size_t total = sizeof(long long) * sol::kProfCtas * sol::kProfRoles * sol::kProfSlots;
  const size_t want = sizeof(long long) * (size_t)n_values;
  return (int)cudaMemcpyFromSymbol(host_out, sol::g_prof, want < total ? want : total);
}
namespace sol {
#endif

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
