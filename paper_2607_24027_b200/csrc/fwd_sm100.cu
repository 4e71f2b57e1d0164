// Sol-Attn fused forward (Algorithm 1) for sm_100a: TMA + tcgen05.mma + TMEM.
//
// Persistent kernel, one CTA of 384 threads per SM, compiled for d in {64, 128} and
// block_q = block_k in {64, 128}.  A CTA owns one query block at a time and is split into warp
// roles that talk through mbarriers:
//
//   router   (warp 8)  pulls (head, query block) work items from a global counter and walks the
//                      pooled keys in chunks of `block` blocks.  For every block it evaluates the
//                      proxy s_ij = scale * Qbar_i . KC_j (Eq. 3) in fp32 and compares it with
//                      tau_i (Eq. 4).  The decision only ever lives in a small shared-memory
//                      record (flat list of tile descriptors + per-column bias); nothing of the
//                      proxy map goes to global memory.
//   producer (warp 9, one lane) reads the records and issues TMA loads: one approximate tile per
//                      chunk (KC chunk, mean-V chunk) and K_j / V_j ONLY for routed blocks.
//   mma      (warps 10, 11) issue tcgen05.mma: warp 10 the score GEMMs S = Q K^T, warp 11 the value
//                      GEMMs O += P V; each warp runs in lockstep and one elected lane issues.  S
//                      goes to one of two TMEM score buffers, so the scores of tile g+1 are
//                      computed while tile g is in softmax.
//   softmax  (warps 0-3 and 4-7) two warpgroups; thread = query row; group h owns key columns
//                      [block/2 * h, block/2 * (h+1)) of EVERY tile and keeps its own running
//                      (m_h, l_h) and its own accumulator O_h in TMEM; the two partial results are
//                      merged when the query block is finished.  Both branches of the method
//                      update the same state: an approximate tile is an ordinary tile whose
//                      columns carry the bias log2(n_j) (Eqs. 9-10: multiplicity n_j in the
//                      denominator, mean value times n_j in the numerator) or -inf for routed /
//                      padded columns.  O_h is rescaled lazily, only when the running maximum
//                      grows by more than 2^8.
//
// The query tile of the MMAs always has 128 rows (the M of a one-CTA tcgen05.mma at full rate);
// with 64-token blocks its upper 64 rows belong to the next query block, take part in the
// arithmetic and are never stored.
//
// TMEM (512 columns): S0 [0, block)  S1 [block, 2 block)  O0 [256, 256 + d)  O1 [256 + d, 256 + 2 d);
// P_h (bf16) of a tile overwrites the start of group h's half of that tile's S buffer.
//
// Every mbarrier wait is bounded: when one expires the CTA records SOL_ERR_DEVICE_TIMEOUT in the
// workspace status word, all roles drain, TMEM is released and the kernel returns.
#include <type_traits>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "tmap.cuh"

namespace sol {
namespace {

using namespace ptx;

constexpr int kRowsQ = 128;                      // rows of the query tile fed to the tensor core
constexpr int kThreads = 384;
constexpr int kKStages = 2;                      // ring of K tiles
constexpr int kVStages = 2;                      // ring of V tiles (its own ring: the score GEMMs run ahead of P V)
constexpr int kGroup = 32;                       // pooled keys scored per router step (one per lane)
constexpr int kRecords = 4;                      // ring of routing records
constexpr int kWarpRouter = 8, kWarpProducer = 9, kWarpQK = 10;   // warp 11 issues P V
constexpr int kTmemCols = 512;
constexpr int kTmemS = 0, kTmemO = 256;
constexpr float kRescaleThreshold = 8.0f;        // log2 units

// Compile-time shape of one kernel instance.
template <int D, int BLK>
struct Cfg {
  static constexpr int kD = D;                     // head dimension
  static constexpr int kBlk = BLK;                 // block_q = block_k = key columns of a tile
  static constexpr int kHalf = BLK / 2;            // key columns per softmax warpgroup
  static constexpr int kBoxes = D / 64;            // 64-channel TMA boxes per tile row
  static constexpr int kQBytes = kRowsQ * D * 2;   // the query tile
  static constexpr int kTileBytes = BLK * D * 2;   // one K-like or V-like tile
  static constexpr int kQBoxBytes = kRowsQ * 128;  // one box of the query tile (64 channels x 128 rows)
  static constexpr int kBoxBytes = BLK * 128;      // one box of a K-like / V-like tile
  static_assert(D == 64 || D == 128, "head dimension");
  static_assert(BLK == 64 || BLK == 128, "block size");
};

// The router turns every chunk of `block` key blocks into a record: a flat list of tile descriptors
// that the other roles only have to read.  A descriptor is (row coordinate << 5) | flags; the
// coordinate is the first key row of an exact tile or the first pooled row of an approximate one.
constexpr uint32_t kTileApprox = 1;      // approximate-branch tile (pooled keys / mean values)
constexpr uint32_t kTileFirst = 2;       // first tile of its work item: Q_i is loaded, accumulators start afresh
constexpr uint32_t kTileEnd = 4;         // not a tile: the work item ends here
constexpr uint32_t kTileEmptyItem = 8;   // on an end entry: the item had no tile at all
constexpr uint32_t kDescStop = 0xffffffffu, kDescAbort = 0xfffffffeu, kDescNone = 0xfffffffdu;

template <class C>
struct alignas(16) Record {
  float bias[C::kBlk];          // approximate-tile column bias: log2(n_j) / (scale * log2 e), or -inf
  int32_t work;                 // bh * Nq + i, or -1: no more work
  int32_t b, h;                 // batch and head of the work item
  int32_t q_row;                // first query row of the work item
  int16_t first, end;           // descriptors [first, end) are valid (slot 0 is kept for the approximate tile)
  uint32_t desc[C::kBlk + 2];
};

template <class C>
struct Shared {
  float kc_stage[2][kGroup * C::kD];   // router: fp32 pooled keys of the group being scored / the next one
  float qbar_s[C::kD];                 // router: pooled query of the current work item
  Record<C> rec[kRecords];
  float2 ml[2][kRowsQ];         // (m_h, l_h) exchange between the softmax warpgroups
  uint64_t rec_full[kRecords], rec_empty[kRecords];
  uint64_t k_full[kKStages], k_empty[kKStages], v_full[kVStages], v_empty[kVStages];
  uint64_t q_full, q_empty;
  uint64_t s_full[2], p_full[2][2], pv_done[2];   // indexed by score buffer (and warpgroup)
  uint64_t x_full;              // rendezvous of the two softmax warpgroups at the end of a work item
  uint64_t o_free;              // all 8 softmax warps have read both accumulators of the finished work item
  uint64_t kc_full[2];          // router staging buffers filled
  uint64_t mma_drain[2];        // abort path only: all MMAs issued by a role have retired
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
  const uint8_t* forced;        // [Nk] or null: key blocks always routed to the exact branch
  Strides st;                   // layout of q, k, v, out
  int rows_inner;               // coordinate order of the q/k/v tensor maps: (c, row, h, b) or (c, h, row, b)
  long long wait_limit;         // SM clocks after which a bounded wait gives up
  int withhold_tile;            // test hook: >= 0: the P V role leaves out the completion signal of this tile
  int out_aligned32;            // every output row piece starts on a 32-byte boundary (32-byte stores are legal)
};

template <class S>
__device__ __forceinline__ void flag_abort(S& sm, const Params& p, int where) {
  sm.abort_flag = 1;
  atomicExch(p.status + kStatusDevice, (int)SOL_ERR_DEVICE_TIMEOUT);
  atomicCAS(p.status + kStatusDetail, 0, where);     // keep the first place that gave up
}

}  // namespace
}  // namespace sol

// Every role has `sm` and `wait_limit` in scope; WAIT is a bounded wait on one of its barriers.
#if defined(SOL_PROFILE) || defined(SOL_ITEMTRACE)
#include "fwd_sm100_prof.cuh"
#endif
#ifdef SOL_PROFILE
#define WAIT(bar, parity, slot) SOL_WAIT(bar, parity, slot)
#else
#define WAIT(bar, parity, slot) mbar_wait((bar), (parity), &sm.abort_flag, wait_limit)
#define PROF_DECL
#define PROF_COUNT(slot)
#define PROF_FLUSH(role)
#define PROF_ACC(slot) nullptr
#define PROF_T0
#define PROF_ADD(slot)
#endif
#ifndef SOL_ITEMTRACE
#define ITRACE(item, slot)
#define ITRACE_VAL(item, slot, val)
#define CTATRACE(slot, val)
#endif

namespace sol {
namespace {

// ------------------------------------------------------------------------------------------------
// Every consumer role (producer, the two MMA warps, both softmax warpgroups) walks the record
// ring with a cursor of its own and sees the same flat stream of descriptors.
template <class C>
struct Cursor {
  uint32_t n_rec = 0;
  int e = 0, end = 0;
  const Record<C>* rec = nullptr;   // the open record (valid until the next call)
};

// `release` is called when the cursor is done with a record (arrives on rec_empty as appropriate
// for the role).  Returns kDescStop at the end of the stream, kDescAbort when a bounded wait
// expired and, with block = false, kDescNone when the next record has not been written yet.
template <class C, class Release>
__device__ __forceinline__ uint32_t next_desc(Shared<C>& sm, Cursor<C>& c, long long wait_limit, long long* wait_acc,
                                              Release release, bool block = true) {
  for (;;) {
    if (c.e < c.end) return c.rec->desc[c.e++];
    if (c.rec) {
      release(c.n_rec % kRecords);
      c.rec = nullptr;
      ++c.n_rec;
    }
    const uint32_t r = c.n_rec % kRecords;
    if (!block && !mbar_try_wait(&sm.rec_full[r], (c.n_rec / kRecords) & 1)) return kDescNone;
#ifdef SOL_PROFILE
    const long long t = clock64();
#endif
    const bool ok = mbar_wait(&sm.rec_full[r], (c.n_rec / kRecords) & 1, &sm.abort_flag, wait_limit);
#ifdef SOL_PROFILE
    if (wait_acc) *wait_acc += clock64() - t;
#endif
    if (!ok) return kDescAbort;
    if (sm.rec[r].work < 0) return kDescStop;        // stays on this record: every further call stops too
    c.rec = &sm.rec[r];
    c.e = c.rec->first;
    c.end = c.rec->end;
  }
}

// ------------------------------------------------------------------------------------------------
// router: one warp
// kFromMask: the decisions were taken by the routing pre-pass and are read back from the mask (one bit per
// (query block, key block)) instead of being scored here.
template <class C, bool kFromMask>
__device__ void router_role(Shared<C>& sm, const Params& p, int lane) {
  constexpr int kD = C::kD, kBlk = C::kBlk, kPieces = C::kD / 4;   // 16-byte pieces per pooled key
  const unsigned full = 0xffffffffu;
  const long long wait_limit = p.wait_limit;
  uint32_t n_rec = 0, n_copy = 0, n_use = 0;   // records written; staging copies issued / consumed
  uint32_t n_item = 0;
  const int n_chunks = ceil_div(p.Nk, kBlk);
  const int mask_words = ceil_div(p.Nk, 32);
  const float inv_sl2 = 1.f / (p.scale * 1.4426950408889634f);   // biases are stored in raw-score units
  constexpr bool from_mask = kFromMask;
  const float bias_full = log2f((float)kBlk) * inv_sl2;                          // log2 n_j of a full block ...
  const float bias_last = log2f((float)(p.N - (p.Nk - 1) * kBlk)) * inv_sl2;     // ... and of the ragged last one
  bool alive = true;
  PROF_DECL
  if (lane == 0) CTATRACE(0, prof::gtimer());
  while (alive) {
    int w = 0;
    if (lane == 0) w = atomicAdd(p.status + kStatusTileCounter, 1);
    w = __shfl_sync(full, w, 0);
    if (w >= p.total_work) break;
    if (lane == 0) ITRACE(n_item, 0);
    const int bh = w / p.Nq, i = w - bh * p.Nq;
    // the pooled query of this work item goes to shared memory (one 16-byte piece per lane)
    float tau_i = 0.f;
    if (p.mode != SOL_MODE_DENSE && !from_mask) {
      __syncwarp();
      if (lane < kPieces)
        reinterpret_cast<float4*>(sm.qbar_s)[lane] =
            __ldg(reinterpret_cast<const float4*>(p.qbar + ((size_t)bh * p.Nq + i) * kD) + lane);
      tau_i = p.tau[(size_t)bh * p.Nq + i];
      __syncwarp();
    }
    const float* kc_head = p.kc + (size_t)bh * p.Nk * kD;
    int count = 0;
    bool item_has_tiles = false;
    // Bulk-copy one group of 32 pooled keys (contiguous in memory) into a staging buffer;
    // the copy of group n+1 is in flight while group n is scored.
    auto stage_group = [&](int jb) {
      if (p.mode == SOL_MODE_DENSE || from_mask || jb >= p.Nk) return;
      __syncwarp();                                  // every lane is done reading this buffer
      if (lane == 0) {
        const uint32_t buf = n_copy & 1;
        const uint32_t bytes = (uint32_t)min(kGroup, p.Nk - jb) * kD * 4;
        fence_proxy_async_smem();
        mbar_arrive_expect_tx(&sm.kc_full[buf], bytes);
        bulk_load_1d(sm.kc_stage[buf], kc_head + (size_t)jb * kD, bytes, &sm.kc_full[buf]);
      }
      ++n_copy;
    };
    stage_group(0);
    for (int t = 0; t < n_chunks; ++t) {
      Record<C>& rec = sm.rec[n_rec % kRecords];
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
        } else if (from_mask) {
          sel = (j < p.Nk) && ((p.mask_out[(size_t)w * mask_words + jbase / 32] >> lane) & 1u);
        } else {
          // lane l scores pooled key jbase + l against the staged rows.  Lane l starts at 16-byte
          // piece l of its row and of the query and walks round, so that the lanes spread over the
          // shared-memory bank groups although the rows are a multiple of 128 bytes apart.
          float dot = 0.f;
          if (jbase < p.Nk) {
            const uint32_t buf = n_use & 1;
            if (!WAIT(&sm.kc_full[buf], (n_use >> 1) & 1, 1)) {                         // prof 1: pooled keys not staged
              if (lane == 0) flag_abort(sm, p, 102);
              alive = false;
              break;
            }
            ++n_use;
            stage_group(jbase + kGroup);              // next group of this work item, if any
            const float4* row = reinterpret_cast<const float4*>(sm.kc_stage[buf] + lane * kD);
            const float4* qv = reinterpret_cast<const float4*>(sm.qbar_s);
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
            for (int c = 0; c < kPieces; ++c) {
              const int piece = (c + lane) & (kPieces - 1);
              const float4 kk = row[piece];
              const float4 qq = qv[piece];
              a0 = fmaf(qq.x, kk.x, a0);
              a1 = fmaf(qq.y, kk.y, a1);
              a2 = fmaf(qq.z, kk.z, a2);
              a3 = fmaf(qq.w, kk.w, a3);
            }
            dot = (a0 + a1) + (a2 + a3);
          }
          sel = (j < p.Nk) && (p.scale * dot > tau_i);
          if (p.forced && j < p.Nk && p.forced[j]) sel = true;
        }
        const unsigned m = __ballot_sync(full, sel);
        const bool valid = j < p.Nk;
        any_unselected |= (valid && !sel);
        rec.bias[g * 32 + lane] = (valid && !sel) ? (j == p.Nk - 1 ? bias_last : bias_full) : -INFINITY;
        if (sel) rec.desc[1 + n_sel + __popc(m & ((1u << lane) - 1u))] = (uint32_t)(j * kBlk) << 5;
        n_sel += __popc(m);
        if (p.mask_out && !from_mask && lane == 0 && jbase < p.Nk) p.mask_out[(size_t)w * mask_words + jbase / 32] = m;
      }
      if (!alive) break;
      any_unselected = __any_sync(full, any_unselected);
      count += n_sel;
      const bool has_approx = p.mode == SOL_MODE_SOL && any_unselected;
      const int first = has_approx ? 0 : 1;
      int end = 1 + n_sel;                   // n_sel <= block
      __syncwarp();
      if (lane == 0) {
        rec.work = w;
        rec.b = bh / p.st.H;
        rec.h = bh - rec.b * p.st.H;
        rec.q_row = i * kBlk;
        if (has_approx) rec.desc[0] = ((uint32_t)j0 << 5) | kTileApprox;
        if (!item_has_tiles && end > first) rec.desc[first] |= kTileFirst;
        if (t == n_chunks - 1) rec.desc[end] = kTileEnd | ((item_has_tiles || end > first) ? 0u : kTileEmptyItem);
        rec.first = (int16_t)first;
        rec.end = (int16_t)(end + (t == n_chunks - 1 ? 1 : 0));
      }
      item_has_tiles |= end > first;
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.rec_full[n_rec % kRecords]);
      if (lane == 0 && t == 0) ITRACE(n_item, 1);
      if (lane == 0 && t == n_chunks - 1) ITRACE(n_item, 2);
      ++n_rec;
    }
    if (alive && lane == 0 && p.counts) p.counts[w] = count;
    ++n_item;
  }
  if (lane == 0) { CTATRACE(1, prof::gtimer()); CTATRACE(2, (long long)n_item); }
  PROF_FLUSH(0);
  if (!alive) {
    // let a staging copy that is still in flight land before the CTA's shared memory goes away
    int never = 0;                                   // this drain must not be cut short by the abort flag
    for (; n_use != n_copy; ++n_use) mbar_wait(&sm.kc_full[n_use & 1], (n_use >> 1) & 1, &never, wait_limit);
  }
  // end-of-stream record
  if (alive) {
    if (mbar_wait(&sm.rec_empty[n_rec % kRecords], ((n_rec / kRecords) & 1) ^ 1, &sm.abort_flag, wait_limit)) {
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
// producer: one thread.  K and V tiles have rings of their own, and the K loads run kLead tiles
// ahead of the V loads: that is the order in which the slots come free (a K slot when its score
// GEMM retires, a V slot a softmax pass and a P V later), so an in-order thread seldom waits for a
// slot while another load could go.
template <class C>
__device__ void producer_role(Shared<C>& sm, const Params& p, unsigned char* sQ, unsigned char* sKV,
                              const CUtensorMap* tm_q, const CUtensorMap* tm_k, const CUtensorMap* tm_v,
                              const CUtensorMap* tm_kc, const CUtensorMap* tm_vm) {
  constexpr int kLead = 2;
  constexpr int kTileBytes = C::kTileBytes;
  const long long wait_limit = p.wait_limit;
  uint32_t n_k = 0, n_v = 0, n_item = 0;
  Cursor<C> cur_k, cur_v;
  PROF_DECL
  // pooled = true: KC / mean-V operands, dense [B*H][Nk][d]; else q, k, v in the caller's layout.
  // A tile is C::kBoxes boxes of 64 channels, each kBox bytes long in shared memory.
  auto load_tile = [&](auto bytes_c, auto box_c, const CUtensorMap* tm, uint64_t* full, unsigned char* dst, int row,
                       const Record<C>* rec, bool pooled) {
    constexpr int kBytes = decltype(bytes_c)::value, kBox = decltype(box_c)::value;
    mbar_arrive_expect_tx(full, kBytes);
    const bool rows_inner = pooled || p.rows_inner;
    const int c1 = rows_inner ? row : rec->h, c2 = rows_inner ? rec->h : row;
    tma_load_4d(dst, tm, full, 0, c1, c2, rec->b);
    if constexpr (C::kBoxes == 2) tma_load_4d(dst + kBox, tm, full, 64, c1, c2, rec->b);
  };
  using QBytes = std::integral_constant<int, C::kQBytes>;
  using QBox = std::integral_constant<int, C::kQBoxBytes>;
  using TBytes = std::integral_constant<int, C::kTileBytes>;
  using TBox = std::integral_constant<int, C::kBoxBytes>;
  auto release = [&](uint32_t r) { mbar_arrive(&sm.rec_empty[r]); };
  bool k_end = false, have_k = false, ok = true;
  uint32_t dk = 0;
  for (;;) {
    // K side (and Q): up to kLead tiles ahead of the V side
    while (!k_end && (int)(n_k - n_v) < kLead) {
      if (!have_k) {
        // never sleep on the router while a V load is owed: the router may itself be waiting for
        // the V cursor to hand a record back
        dk = next_desc(sm, cur_k, wait_limit, PROF_ACC(0), release, n_k == n_v);      // prof 0: no record yet
        if (dk == kDescNone) break;
        if (dk == kDescAbort) { ok = false; break; }
        if (dk == kDescStop) { k_end = true; break; }
        have_k = true;
      }
      if (dk & kTileEnd) { have_k = false; continue; }
      if (dk & kTileFirst) {
        // Q_i for this work item.  The slot frees when the previous item's last score GEMM
        // retires; until then serve the V side.
        const uint32_t par = (n_item & 1) ^ 1;
        if (n_k != n_v && !mbar_try_wait(&sm.q_empty, par)) break;
        if (!WAIT(&sm.q_empty, par, 2)) { ok = false; break; }                  // prof 2: Q slot busy
        load_tile(QBytes{}, QBox{}, tm_q, &sm.q_full, sQ, cur_k.rec->q_row, cur_k.rec, false);
        ++n_item;
        dk &= ~kTileFirst;
      }
      have_k = false;
      const uint32_t s = n_k % kKStages;
      if (!WAIT(&sm.k_empty[s], ((n_k / kKStages) & 1) ^ 1, 1)) { ok = false; break; }   // prof 1: K ring full
      {
        PROF_T0
        load_tile(TBytes{}, TBox{}, (dk & kTileApprox) ? tm_kc : tm_k, &sm.k_full[s], sKV + (size_t)s * kTileBytes,
                  (int)(dk >> 5), cur_k.rec, (dk & kTileApprox) != 0);
        PROF_ADD(4)                                                                    // prof 4: issuing K copies
      }
      ++n_k;
    }
    if (!ok) break;
    if (n_k == n_v) {
      if (k_end) break;
      continue;
    }
    // V side: the oldest tile whose K is already on its way
    uint32_t dv;
    {
      PROF_T0
      do {
        dv = next_desc(sm, cur_v, wait_limit, nullptr, release);
      } while (dv < kDescNone && (dv & kTileEnd));
      PROF_ADD(6)                                                                      // prof 6: V cursor
    }
    if (dv >= kDescNone) { ok = false; break; }          // cannot end before the K side did
    const uint32_t s = n_v % kVStages;
    if (!WAIT(&sm.v_empty[s], ((n_v / kVStages) & 1) ^ 1, 3)) { ok = false; break; }     // prof 3: V ring full
    {
      PROF_T0
      load_tile(TBytes{}, TBox{}, (dv & kTileApprox) ? tm_vm : tm_v, &sm.v_full[s],
                sKV + (size_t)(kKStages + s) * kTileBytes, (int)(dv >> 5), cur_v.rec, (dv & kTileApprox) != 0);
      PROF_ADD(5)                                                                      // prof 5: issuing V copies
    }
    ++n_v;
  }
  if (ok) {
    // the V cursor still has to hand back the records that hold no further tile
    for (;;) {
      const uint32_t dv = next_desc(sm, cur_v, wait_limit, nullptr, release);
      if (dv >= kDescNone) break;
    }
  } else {
    flag_abort(sm, p, 200);
  }
  PROF_FLUSH(1);
  if (sm.abort_flag) {
    // let copies that are still in flight land before the CTA's shared memory goes away
    int never = 0;                                   // this drain must not be cut short by the abort flag
    if (n_item > 0) mbar_wait(&sm.q_full, (n_item - 1) & 1, &never, wait_limit);
    for (uint32_t back = 0; back < kKStages && back < n_k; ++back) {
      const uint32_t n = n_k - 1 - back;
      mbar_wait(&sm.k_full[n % kKStages], (n / kKStages) & 1, &never, wait_limit);
    }
    for (uint32_t back = 0; back < kVStages && back < n_v; ++back) {
      const uint32_t n = n_v - 1 - back;
      mbar_wait(&sm.v_full[n % kVStages], (n / kVStages) & 1, &never, wait_limit);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// MMA issue is split over two single-thread roles so that neither the waits nor the scalar
// bookkeeping of one kind of MMA delays the other; the tensor pipe arbitrates between them and all
// ordering is carried by the mbarriers.
//
// Shared-memory descriptors: the upper word is constant (stride 1024 B between 8-row groups,
// descriptor version, 128-byte swizzle); the lower word is (address >> 4) | (leading offset >> 4) << 16.
__device__ __forceinline__ uint64_t desc_from_lo(uint32_t lo) {
  constexpr uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
  return ((uint64_t)hi << 32) | lo;
}

// Abort path of an MMA-issuing role: TMEM must not be released while MMAs are still writing to it, so
// the role asks for a completion signal behind everything it has issued and waits for it (bounded).
template <class C>
__device__ __forceinline__ void drain_mmas(Shared<C>& sm, uint64_t* bar, bool leader, long long wait_limit) {
  if (leader) mma_commit(bar);
  int never = 0;
  mbar_wait(bar, 0, &never, wait_limit);
}

// S_b = Q K^T (warp 10)
template <class C>
__device__ void mma_qk_role(Shared<C>& sm, const Params& p, unsigned char* sQ, unsigned char* sKV, uint32_t tmem) {
  constexpr int kD = C::kD, kBlk = C::kBlk, kTileBytes = C::kTileBytes;
  const long long wait_limit = p.wait_limit;
  const uint32_t idesc_qk = make_idesc_bf16(kRowsQ, kBlk, false, false);
  const uint32_t q_lo = (smem_addr(sQ) >> 4) | (1u << 16);
  const uint32_t kv_lo = (smem_addr(sKV) >> 4) | (1u << 16);
  uint32_t n_item = 0, g = 0;
  uint32_t slot = 0, slot_parity = 0;          // ring position of K(g)
  Cursor<C> cur;
  PROF_DECL
  // The whole warp runs this role in lockstep and one elected lane issues: with warp-uniform control
  // flow and operands the compiler keeps descriptors and addresses in uniform registers, where the
  // MMA instruction wants them, instead of moving them over from a single divergent lane's registers.
  const bool leader = elect_one();
  auto release = [&](uint32_t r) { if (leader) mbar_arrive(&sm.rec_empty[r]); };
  bool ok = true;
  for (;;) {
    const uint32_t dsc = next_desc(sm, cur, wait_limit, PROF_ACC(0), release);        // prof 0: no record yet
    if (dsc == kDescAbort) { ok = false; break; }
    if (dsc == kDescStop) break;
    if (dsc & kTileEnd) {                         // every MMA that reads Q_i has been issued
      if (!(dsc & kTileEmptyItem) && leader) mma_commit(&sm.q_empty);
      continue;
    }
    const bool it_first = (dsc & kTileFirst) != 0;
    if (it_first) {
      if (leader) ITRACE(n_item, 3);
      if (!WAIT(&sm.q_full, n_item & 1, 1)) { ok = false; break; }                    // prof 1: Q not loaded
      ++n_item;
    }
    const uint32_t b = g & 1;
    if (!WAIT(&sm.k_full[slot], slot_parity, 2)) { ok = false; break; }               // prof 2: K not loaded
    if (g >= 2) {
      // P overwrites S: the P V of tile g-2 must have read P out of this buffer
      if (!WAIT(&sm.pv_done[b], ((g - 2) >> 1) & 1, 3)) { ok = false; break; }        // prof 3: score buffer busy
    }
    tc_fence_after();
    {
      PROF_T0
      const uint32_t k_lo = kv_lo + slot * (kTileBytes >> 4);
      const uint32_t d_tmem = tmem + kTmemS + b * kBlk;
#pragma unroll
      for (int ks = 0; ks < kD / 16; ++ks) {
        // K-step ks: 16 channels = 32 bytes inside box ks / 4
        const uint32_t off_q = ((ks / 4) * C::kQBoxBytes + (ks % 4) * 32) >> 4;
        const uint32_t off_k = ((ks / 4) * C::kBoxBytes + (ks % 4) * 32) >> 4;
        const uint64_t da = desc_from_lo(q_lo + off_q), db = desc_from_lo(k_lo + off_k);
        if (leader) mma_ss(d_tmem, da, db, idesc_qk, ks > 0);
      }
      if (leader) {
        mma_commit(&sm.k_empty[slot]);
        mma_commit(&sm.s_full[b]);
      }
      PROF_ADD(6)                                                                      // prof 6: issuing Q K^T
      if (it_first && leader) ITRACE(n_item - 1, 4);
    }
    ++g;
    if (++slot == kKStages) { slot = 0; slot_parity ^= 1; }
  }
  if (!ok && leader) flag_abort(sm, p, 300);
  __syncwarp();
  if (sm.abort_flag) drain_mmas(sm, &sm.mma_drain[0], leader, wait_limit);
  if (leader) PROF_FLUSH(2);
}

// O_h (+)= P_h V[half h of the tile's keys], h = 0, 1 (warp 11)
template <class C>
__device__ void mma_pv_role(Shared<C>& sm, const Params& p, unsigned char* sKV, uint32_t tmem) {
  constexpr int kD = C::kD, kBlk = C::kBlk, kHalf = C::kHalf, kTileBytes = C::kTileBytes;
  const long long wait_limit = p.wait_limit;
  const uint32_t idesc_pv = make_idesc_bf16(kRowsQ, kD, false, true);
  // V is the MN-major operand: its 64-channel boxes are C::kBoxBytes apart (leading offset), groups of
  // 8 key rows 1024 bytes apart; a K-step of 16 keys advances the start by 2048 bytes.
  const uint32_t kv_lo = (smem_addr(sKV + kKStages * kTileBytes) >> 4) | ((uint32_t)(C::kBoxBytes >> 4) << 16);
  uint32_t g = 0, n_item = 0;
  uint32_t slot = 0, slot_parity = 0;          // ring position of V(g)
  Cursor<C> cur;
  const bool leader = elect_one();             // warp-uniform role, one issuing lane (see mma_qk_role)
  auto release = [&](uint32_t r) { if (leader) mbar_arrive(&sm.rec_empty[r]); };
  bool ok = true;
  for (;;) {
    const uint32_t dsc = next_desc(sm, cur, wait_limit, nullptr, release);
    if (dsc == kDescAbort) { ok = false; break; }
    if (dsc == kDescStop) break;
    if (dsc & kTileEnd) continue;
    const uint32_t b = g & 1;
    if (!mbar_wait(&sm.v_full[slot], slot_parity, &sm.abort_flag, wait_limit)) { ok = false; break; }
    const uint32_t v_lo = kv_lo + slot * (kTileBytes >> 4);
    const uint32_t acc_first = (dsc & kTileFirst) ? 0u : 1u;
    if ((dsc & kTileFirst) && n_item++ > 0) {
      // the first P V of a work item overwrites O0 / O1: the previous item's merge must have read them
      if (!mbar_wait(&sm.o_free, (n_item - 2) & 1, &sm.abort_flag, wait_limit)) { ok = false; break; }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      if (!mbar_wait(&sm.p_full[h][b], (g >> 1) & 1, &sm.abort_flag, wait_limit)) { ok = false; break; }
      tc_fence_after();
#pragma unroll
      for (int ks = 0; ks < kHalf / 16; ++ks) {
        const uint32_t d_o = tmem + kTmemO + h * kD;
        const uint32_t a_p = tmem + kTmemS + b * kBlk + h * kHalf + ks * 8;
        const uint32_t acc = ks > 0 ? 1u : acc_first;
        const uint64_t dv = desc_from_lo(v_lo + ((h * (kHalf * 128) + ks * 2048) >> 4));
        if (leader) mma_ts(d_o, a_p, dv, idesc_pv, acc);
      }
    }
    if (!ok) break;
    if (leader) {
      mma_commit(&sm.v_empty[slot]);
      // (test hook: a withheld completion signal makes the bounded waits on it run out)
      if ((int)g != p.withhold_tile) mma_commit(&sm.pv_done[b]);
    }
    ++g;
    if (++slot == kVStages) { slot = 0; slot_parity ^= 1; }
  }
  if (!ok && leader) flag_abort(sm, p, 301);
  __syncwarp();
  if (sm.abort_flag) drain_mmas(sm, &sm.mma_drain[1], leader, wait_limit);
}

// ------------------------------------------------------------------------------------------------
// softmax + correction + epilogue: two warpgroups of 128 threads; thread = query row, warpgroup h
// owns key columns [kHalf h, kHalf (h+1)) of every tile.
template <int N>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t* r) {   // N columns, N a multiple of 32
#pragma unroll
  for (int c = 0; c < N; c += 32) tmem_ld_32x32b_x32(taddr + c, *reinterpret_cast<uint32_t(*)[32]>(r + c));
}

template <class C>
__device__ void softmax_role(Shared<C>& sm, const Params& p, uint32_t tmem, int h, int warp_in_group, int lane) {
  constexpr int kD = C::kD, kBlk = C::kBlk, kHalf = C::kHalf;
  constexpr int kOutCh = kD / 2;                             // output channels written by one warpgroup
  const unsigned full = 0xffffffffu;
  const long long wait_limit = p.wait_limit;
  const uint32_t lane_base = tmem + ((uint32_t)(warp_in_group * 32) << 16);
  const uint32_t t_o = lane_base + kTmemO + h * kD;          // this group's accumulator
  const uint32_t t_o_other = lane_base + kTmemO + (1 - h) * kD;
  const int row = warp_in_group * 32 + lane;
  const float sl2 = p.scale * 1.4426950408889634f;
  uint32_t g = 0, n_merge = 0;
  uint32_t n_item = 0, g_item0 = 0;        // item trace only
  float m_used = -INFINITY, l = 0.f;
  Cursor<C> cur;
  PROF_DECL
  auto release = [&](uint32_t r) {
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.rec_empty[r]);
  };
  // A wait that gives up must give up for the whole warp: the loop holds warp-synchronising
  // operations (TMEM loads and stores, votes), so the lanes leave together or not at all.
#define SWAIT(bar, parity, slot) __all_sync(full, WAIT(bar, parity, slot))
  // The next descriptor of the open record is read from shared memory while the current tile is being
  // worked on, so that the read's latency is off the path from one tile to the next.
  bool peeked = false;
  uint32_t dsc_peek = 0;
  for (;;) {
    uint32_t dsc;
    if (peeked) {
      dsc = dsc_peek;
      ++cur.e;
    } else {
      dsc = next_desc(sm, cur, wait_limit, PROF_ACC(0), release);                     // prof 0: no record yet
      if (dsc == kDescAbort) { flag_abort(sm, p, 400); break; }
      if (dsc == kDescStop) break;
    }
    peeked = cur.e < cur.end;
    if (peeked) dsc_peek = cur.rec->desc[cur.e];
    const bool first = (dsc & kTileFirst) != 0;

    if (!(dsc & kTileEnd)) {
      const uint32_t b = g & 1;
      const uint32_t t_s = lane_base + kTmemS + b * kBlk + h * kHalf;
      const bool approx = (dsc & kTileApprox) != 0;
      const int cols_valid = approx ? kBlk : min(kBlk, p.N - (int)(dsc >> 5));
      const bool general = approx || cols_valid < kBlk;
      // (no vote on this wait, the one wait of every tile: the 32 lanes poll the same barrier, abort flag
      //  and clock in lockstep and leave the loop together; the rarer waits below are made uniform by a vote)
      if (!WAIT(&sm.s_full[b], (g >> 1) & 1, 1)) { flag_abort(sm, p, 401); break; }   // prof 1: S not ready
      tc_fence_after();
      if (first && warp_in_group == 0 && lane == 0) { ITRACE(n_item, h ? 11 : 5); g_item0 = g; }
      // ---- this group's half row of S (kHalf fp32) into registers with one wait
      uint32_t sr[kHalf];
      PROF_T0
      tmem_ld_cols<kHalf>(t_s, sr);
      tmem_ld_wait();
      PROF_ADD(7)                                                                      // prof 7: loading S
      if (general) {
        // bring the rare tiles (approximate chunk, ragged last block) to the common form
        // logit = sl2 * x by folding the column bias into x; -inf marks masked columns
        if (approx) {
          const float4* bias4 = reinterpret_cast<const float4*>(&cur.rec->bias[h * kHalf]);
#pragma unroll
          for (int c = 0; c < kHalf / 4; ++c) {
            const float4 bb = bias4[c];
            sr[4 * c] = __float_as_uint(__uint_as_float(sr[4 * c]) + bb.x);
            sr[4 * c + 1] = __float_as_uint(__uint_as_float(sr[4 * c + 1]) + bb.y);
            sr[4 * c + 2] = __float_as_uint(__uint_as_float(sr[4 * c + 2]) + bb.z);
            sr[4 * c + 3] = __float_as_uint(__uint_as_float(sr[4 * c + 3]) + bb.w);
          }
        } else {
#pragma unroll
          for (int c = 0; c < kHalf; ++c)
            if (h * kHalf + c >= cols_valid) sr[c] = __float_as_uint(-INFINITY);
        }
      }
      float mx;
      {
        constexpr int kQ = kHalf / 4;
        float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
        for (int c = 0; c < kQ; ++c) {
          m0 = fmaxf(m0, __uint_as_float(sr[c]));
          m1 = fmaxf(m1, __uint_as_float(sr[kQ + c]));
          m2 = fmaxf(m2, __uint_as_float(sr[2 * kQ + c]));
          m3 = fmaxf(m3, __uint_as_float(sr[3 * kQ + c]));
        }
        mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)) * sl2;       // -inf when the whole half is masked
      }
      // ---- running maximum, lazy rescale of O_h
      if (first) {
        m_used = mx;
        l = 0.f;
      } else if (__any_sync(full, mx > m_used + kRescaleThreshold)) {
        const float m_new = fmaxf(m_used, mx);
        const float f = (m_new == -INFINITY) ? 1.f : ex2(m_used - m_new);
        PROF_COUNT(4);                                                                  // prof 4: number of rescales
        // P V of the previous tile must have landed in O_h
        if (!SWAIT(&sm.pv_done[b ^ 1], ((g - 1) >> 1) & 1, 2)) { flag_abort(sm, p, 402); break; }
        tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < kD / 32; ++c) {
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
      // ---- P = exp2(sl2 * S - m) (scaling and row sum as packed fp32 pairs); P (bf16) back to
      //      TMEM over the start of the half
      {
        const float nm = (m_used == -INFINITY) ? 0.f : -m_used;   // a half that has seen nothing yet: all P = 0
        const float2 sl2_2 = make_float2(sl2, sl2), nm2 = make_float2(nm, nm);
        float2 s_a = make_float2(0.f, 0.f), s_b = make_float2(0.f, 0.f);
#pragma unroll
        for (int c = 0; c < kHalf; c += 4) {
          const float2 xa = __ffma2_rn(make_float2(__uint_as_float(sr[c]), __uint_as_float(sr[c + 1])), sl2_2, nm2);
          const float2 xb = __ffma2_rn(make_float2(__uint_as_float(sr[c + 2]), __uint_as_float(sr[c + 3])), sl2_2, nm2);
          const float2 ea = make_float2(ex2(xa.x), ex2(xa.y));
          const float2 eb = make_float2(ex2(xb.x), ex2(xb.y));
          s_a = __fadd2_rn(s_a, ea);
          s_b = __fadd2_rn(s_b, eb);
          __nv_bfloat162 lo = __floats2bfloat162_rn(ea.x, ea.y);
          __nv_bfloat162 hi = __floats2bfloat162_rn(eb.x, eb.y);
          sr[c / 2] = *reinterpret_cast<uint32_t*>(&lo);
          sr[c / 2 + 1] = *reinterpret_cast<uint32_t*>(&hi);
        }
        {
          const float2 t = __fadd2_rn(s_a, s_b);
          l += t.x + t.y;
        }
        if constexpr (kHalf == 64) tmem_st_32x32b_x32(t_s, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
        else tmem_st_32x32b_x16(t_s, *reinterpret_cast<uint32_t(*)[16]>(&sr[0]));
      }
      PROF_ADD(8)                                                                      // prof 8: load + arithmetic
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();                                  // one arrival per warp: 4 instead of 128 on the barrier
      if (lane == 0) mbar_arrive(&sm.p_full[h][b]);
      PROF_ADD(9)                                                                      // prof 9: whole tile
#ifdef SOL_PROFILE
      if (approx) { prof.v[10] += clock64() - prof_t0; ++prof.v[0]; }                  // prof 10 / 0: approximate tiles: cycles / count
#endif
      PROF_COUNT(5);                                                                    // prof 5: tiles
      ++g;
      continue;
    }

    // ---- end of the work item: merge the two partial results, O_i = (w0 O0 + w1 O1) / (w0 l0 + w1 l1)
    const int q_row = cur.rec->q_row;
    const int q_rows = min(kBlk, p.N - q_row);
    __nv_bfloat16* orow = p.out + (size_t)cur.rec->b * (size_t)p.st.batch + (size_t)cur.rec->h * (size_t)p.st.head +
                          (size_t)(q_row + row) * (size_t)p.st.row + h * kOutCh;
    PROF_T0
    if (warp_in_group == 0 && lane == 0) {
      ITRACE(n_item, h ? 12 : 6);
      if (h == 0) ITRACE_VAL(n_item, 10, (long long)(g - g_item0));
    }
    if (!(dsc & kTileEmptyItem)) {
      // the last P V of the item (one commit covers both halves)
      if (!SWAIT(&sm.pv_done[(g - 1) & 1], ((g - 1) >> 1) & 1, 3)) { flag_abort(sm, p, 403); break; }   // prof 3
      tc_fence_after();
      if (h == 0 && warp_in_group == 0 && lane == 0) ITRACE(n_item, 7);
      sm.ml[h][row] = make_float2(m_used, l);
      mbar_arrive(&sm.x_full);
      if (!SWAIT(&sm.x_full, n_merge & 1, 6)) { flag_abort(sm, p, 404); break; }      // prof 6: other group not done
      if (warp_in_group == 0 && lane == 0) ITRACE(n_item, h ? 13 : 8);
      const float2 other = sm.ml[1 - h][row];
      const float m = fmaxf(m_used, other.x);
      const float w_own = (m_used == -INFINITY) ? 0.f : ex2(m_used - m);
      const float w_other = (other.x == -INFINITY) ? 0.f : ex2(other.x - m);
      const float inv = 1.f / (l * w_own + other.y * w_other);
      const float c_own = w_own * inv, c_other = w_other * inv;
      // this thread writes channels [kOutCh h, kOutCh (h+1)) of its row
#pragma unroll 1
      for (int c = 0; c < kOutCh / 32; ++c) {
        uint32_t a[32], bb[32];
        tmem_ld_32x32b_x32(t_o + h * kOutCh + c * 32, a);
        tmem_ld_32x32b_x32(t_o_other + h * kOutCh + c * 32, bb);
        tmem_ld_wait();
        if (c == kOutCh / 32 - 1) {
          // both accumulators are in registers: the next item's first P V may overwrite them
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.o_free);
        }
        if (row < q_rows) {
#pragma unroll
          for (int x = 0; x < 2; ++x) {                 // 32 bytes (16 channels) per store
            uint32_t pw[8];
#pragma unroll
            for (int y = 0; y < 8; ++y) {
              const int e0 = x * 16 + 2 * y;
              // a partial accumulator that never received a tile may hold anything: weight 0 must win
              const float v0 = (w_own > 0.f ? __uint_as_float(a[e0]) * c_own : 0.f) +
                               (w_other > 0.f ? __uint_as_float(bb[e0]) * c_other : 0.f);
              const float v1 = (w_own > 0.f ? __uint_as_float(a[e0 + 1]) * c_own : 0.f) +
                               (w_other > 0.f ? __uint_as_float(bb[e0 + 1]) * c_other : 0.f);
              __nv_bfloat162 hh = __floats2bfloat162_rn(v0, v1);
              pw[y] = *reinterpret_cast<uint32_t*>(&hh);
            }
            if (p.out_aligned32) {
              st_global_v8(orow + c * 32 + x * 16, pw);
            } else {                                    // the interface only asks for 16-byte alignment
              uint4* dst = reinterpret_cast<uint4*>(orow + c * 32 + x * 16);
              dst[0] = make_uint4(pw[0], pw[1], pw[2], pw[3]);
              dst[1] = make_uint4(pw[4], pw[5], pw[6], pw[7]);
            }
          }
        }
      }
      if (warp_in_group == 0 && lane == 0) ITRACE(n_item, h ? 14 : 9);
      ++n_merge;
    } else if (row < q_rows) {
      // a query block that routed nothing in keep-or-drop mode has no attention mass at all
      for (int c = 0; c < kOutCh; c += 8) *reinterpret_cast<uint4*>(orow + c) = make_uint4(0, 0, 0, 0);
    }
    m_used = -INFINITY;
    l = 0.f;
    ++n_item;
    PROF_ADD(2)                                                                        // prof 2: whole epilogue
  }
#undef SWAIT
  if (lane == 0 && warp_in_group == 0 && h == 0) { PROF_FLUSH(3); CTATRACE(3, prof::gtimer()); }
}

template <class C, bool kFromMask>
__global__ void __launch_bounds__(kThreads, 1)
fwd_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_kc,
                 const __grid_constant__ CUtensorMap tm_vm, const Params p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* sQ = base;
  unsigned char* sKV = base + C::kQBytes;
  Shared<C>& sm = *reinterpret_cast<Shared<C>*>(base + C::kQBytes + (kKStages + kVStages) * C::kTileBytes);
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;

  if (threadIdx.x == 0) {
    sm.abort_flag = 0;
    // a record is released by the producer's two cursors, the two MMA warps and the 8 softmax warps
    for (int r = 0; r < kRecords; ++r) { mbar_init(&sm.rec_full[r], 1); mbar_init(&sm.rec_empty[r], 12); }
    for (int s = 0; s < kKStages; ++s) { mbar_init(&sm.k_full[s], 1); mbar_init(&sm.k_empty[s], 1); }
    for (int s = 0; s < kVStages; ++s) { mbar_init(&sm.v_full[s], 1); mbar_init(&sm.v_empty[s], 1); }
    mbar_init(&sm.q_full, 1); mbar_init(&sm.q_empty, 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(&sm.s_full[b], 1);
      mbar_init(&sm.pv_done[b], 1);
      mbar_init(&sm.p_full[0][b], 4);
      mbar_init(&sm.p_full[1][b], 4);
    }
    mbar_init(&sm.x_full, 256); mbar_init(&sm.o_free, 8);
    mbar_init(&sm.kc_full[0], 1); mbar_init(&sm.kc_full[1], 1);
    mbar_init(&sm.mma_drain[0], 1); mbar_init(&sm.mma_drain[1], 1);
    fence_mbar_init();
  }
  if (warp == kWarpProducer && lane == 0) {
    prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v);
    prefetch_tensormap(&tm_kc); prefetch_tensormap(&tm_vm);
  }
  if (warp == 0) { tmem_alloc(&sm.tmem_base, kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp < 8) {
    softmax_role<C>(sm, p, tmem, warp / 4, warp % 4, lane);
  } else if (warp == kWarpRouter) {
    router_role<C, kFromMask>(sm, p, lane);
  } else if (warp == kWarpProducer) {
    if (lane == 0) producer_role<C>(sm, p, sQ, sKV, &tm_q, &tm_k, &tm_v, &tm_kc, &tm_vm);
  } else if (warp == kWarpQK) {
    mma_qk_role<C>(sm, p, sQ, sKV, tmem);
  } else {
    mma_pv_role<C>(sm, p, sKV, tmem);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// Test hook (sol_attn_debug_set_wait): the wait limit and the withheld tile of the following launches.
long long g_wait_limit = kWaitCycles;
int g_withhold_tile = -1;

template <class C>
cudaError_t launch_instance(const Problem& p, const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                            __nv_bfloat16* out, const WsPtrs& ws, const float* tau, int32_t* counts, uint32_t* mask_out,
                            cudaStream_t stream, int* n_launches) {
  CUtensorMap tq, tk, tv, tkc, tvm;
  bool rows_inner = true, pooled_inner = true;
  auto user_map = [&](CUtensorMap* m, const void* base, int box_rows) {
    return make_tmap_bf16_4d(m, base, p.B, p.H, p.N, C::kD, box_rows, p.st.row, p.st.head, p.st.batch, &rows_inner);
  };
  auto pooled_map = [&](CUtensorMap* m, const void* base) {      // dense [B][H][Nk][d]
    return make_tmap_bf16_4d(m, base, p.B, p.H, p.Nk, C::kD, C::kBlk, C::kD, (long long)p.Nk * C::kD,
                             (long long)p.H * p.Nk * C::kD, &pooled_inner);
  };
  if (!user_map(&tq, q, kRowsQ) || !user_map(&tk, k, C::kBlk) || !user_map(&tv, v, C::kBlk) ||
      !pooled_map(&tkc, ws.kcb) || !pooled_map(&tvm, ws.vmb) || !pooled_inner)
    return cudaErrorInvalidValue;
  Params prm{};
  prm.qbar = ws.qbar; prm.kc = ws.kc; prm.tau = tau; prm.out = out; prm.counts = counts; prm.mask_out = mask_out;
  prm.status = ws.status; prm.N = p.N; prm.Nq = p.Nq; prm.Nk = p.Nk; prm.total_work = p.BH * p.Nq;
  prm.mode = p.mode; prm.scale = p.scale; prm.forced = p.forced;
  prm.st = p.st; prm.rows_inner = rows_inner ? 1 : 0;
  prm.wait_limit = g_wait_limit; prm.withhold_tile = g_withhold_tile;
  prm.out_aligned32 = (reinterpret_cast<uintptr_t>(out) % 32 == 0 && (p.st.row * 2) % 32 == 0 && (p.st.head * 2) % 32 == 0 &&
                       (p.st.batch * 2) % 32 == 0) ? 1 : 0;

  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  const size_t smem = 1024 + C::kQBytes + (kKStages + kVStages) * C::kTileBytes + sizeof(Shared<C>);
  const int grid = prm.total_work < sms ? prm.total_work : sms;
  // the pre-pass variant is a kernel of its own, so that the in-kernel router's code is what it is without it
  if (p.routing == SOL_ROUTING_PREPASS && p.mode != SOL_MODE_DENSE) {
    e = cudaFuncSetAttribute(fwd_sm100_kernel<C, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    fwd_sm100_kernel<C, true><<<grid, kThreads, smem, stream>>>(tq, tk, tv, tkc, tvm, prm);
  } else {
    e = cudaFuncSetAttribute(fwd_sm100_kernel<C, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    fwd_sm100_kernel<C, false><<<grid, kThreads, smem, stream>>>(tq, tk, tv, tkc, tvm, prm);
  }
  if (n_launches) *n_launches += 1;
  return cudaGetLastError();
}

}  // namespace

bool fwd_sm100_supports(const Problem& p) {
  return (p.d == 64 || p.d == 128) && p.block_q == p.block_k && (p.block_k == 64 || p.block_k == 128);
}

void fwd_sm100_set_wait(long long wait_cycles, int withhold_tile) {
  g_wait_limit = wait_cycles > 0 ? wait_cycles : kWaitCycles;
  g_withhold_tile = withhold_tile;
}

cudaError_t launch_fwd_sm100(const Problem& p, const __nv_bfloat16* q, const __nv_bfloat16* k,
                             const __nv_bfloat16* v, __nv_bfloat16* out, const WsPtrs& ws, const float* tau,
                             int32_t* counts, uint32_t* mask_out, cudaStream_t stream,
                             int* n_launches) {
  if (!fwd_sm100_supports(p)) return cudaErrorInvalidValue;
  if (p.d == 128 && p.block_k == 128)
    return launch_instance<Cfg<128, 128>>(p, q, k, v, out, ws, tau, counts, mask_out, stream, n_launches);
  if (p.d == 64 && p.block_k == 64)
    return launch_instance<Cfg<64, 64>>(p, q, k, v, out, ws, tau, counts, mask_out, stream, n_launches);
  if (p.d == 128)
    return launch_instance<Cfg<128, 64>>(p, q, k, v, out, ws, tau, counts, mask_out, stream, n_launches);
  return launch_instance<Cfg<64, 128>>(p, q, k, v, out, ws, tau, counts, mask_out, stream, n_launches);
}

}  // namespace sol
