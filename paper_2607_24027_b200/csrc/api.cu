// C ABI of the Sol-Attn CUDA path: argument validation, workspace bookkeeping, launches.
#include <atomic>
#include <mutex>
#include <cmath>
#include <cstdio>
#include <cstdlib>

#include "common.cuh"

namespace {

struct Bound {
  void* ws = nullptr;
  size_t bytes = 0;
  int32_t* counts = nullptr;
};
Bound g_bound;
std::atomic<int64_t> g_launches{0};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Two copy streams and four events per device for the host-buffer entry point, made on first use and
// kept for the life of the process (host-side objects; no device memory is involved).  An event may be
// recorded again and again: a cudaStreamWaitEvent waits for the record that precedes it.
constexpr int kMaxDevices = 64;
std::mutex g_stream_mu;
struct HostPath {
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, copied = nullptr, computed = nullptr, done = nullptr;
};
HostPath g_host[kMaxDevices];

sol_status_t host_path(HostPath* hp) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SOL_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return SOL_ERR_UNSUPPORTED_SHAPE;
  std::lock_guard<std::mutex> lock(g_stream_mu);
  HostPath& h = g_host[dev];
  if (!h.done) {
    if (cudaStreamCreateWithFlags(&h.in, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&h.out, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&h.start, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h.copied, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h.computed, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h.done, cudaEventDisableTiming) != cudaSuccess)
      return SOL_ERR_CUDA;
  }
  *hp = h;
  return SOL_OK;
}

// bytes of one tensor per group of heads on the host path (SOL_ATTN_HOST_GROUP_BYTES may change between calls)
size_t host_group_bytes() {
  size_t want = size_t(64) << 20;                            // about 64 MB per tensor and group
  if (const char* env = getenv("SOL_ATTN_HOST_GROUP_BYTES")) {
    const long long v = atoll(env);
    if (v > 0) want = (size_t)v;
  }
  return want;
}

sol_status_t check_arch() { return sol::check_device_arch(); }

// Shape checks common to every entry point.  `fused` adds the fused kernels' restrictions.
sol_status_t check_shape(int B, int H, int N, int d, int block_q, int block_k, bool fused) {
  if (B <= 0 || H <= 0 || N <= 0 || d <= 0 || block_q <= 0 || block_k <= 0) return SOL_ERR_INVALID_ARG;
  if (d != 64 && d != 128) return SOL_ERR_UNSUPPORTED_SHAPE;
  if (block_q > 1024 || block_k > 1024) return SOL_ERR_UNSUPPORTED_SHAPE;
  if ((long long)B * H > 65535LL) return SOL_ERR_UNSUPPORTED_SHAPE;   // (batch, head) pairs index gridDim.y in the pre-attention kernels
  if (sol::ceil_div(N, block_k) > 65535 || sol::ceil_div(N, block_q) > 65535) return SOL_ERR_UNSUPPORTED_SHAPE;
  if ((long long)B * H * sol::ceil_div(N, block_q) > 0x7fffffffLL) return SOL_ERR_UNSUPPORTED_SHAPE;   // work items are counted in int32
  if (fused && (block_q != block_k || (block_q != 64 && block_q != 128))) return SOL_ERR_UNSUPPORTED_SHAPE;
  return SOL_OK;
}

sol::Problem make_problem(int B, int H, int N, int d, int block_q, int block_k, float beta, float scale, int mode,
                          int estimator = SOL_EST_MOMENTS, const uint8_t* forced = nullptr,
                          int layout = SOL_LAYOUT_BHND) {
  sol::Problem p{};
  p.B = B; p.H = H; p.N = N; p.d = d; p.block_q = block_q; p.block_k = block_k;
  p.BH = B * H;
  p.Nq = sol::ceil_div(N, block_q);
  p.Nk = sol::ceil_div(N, block_k);
  p.scale = scale > 0.f ? scale : 1.0f / std::sqrt((float)d);
  p.beta = beta;
  p.mode = mode;
  p.estimator = estimator;
  p.forced = forced;
  p.st.H = H;
  if (layout == SOL_LAYOUT_BNHD) {
    p.st.row = (long long)H * d; p.st.head = d; p.st.batch = (long long)N * H * d;
  } else {
    p.st.row = d; p.st.head = (long long)N * d; p.st.batch = (long long)H * N * d;
  }
  return p;
}

sol_status_t run_pool(const sol::Problem& p, const void* q, const void* k, const void* v, void* ws_base,
                      cudaStream_t stream) {
  const sol::WsLayout lay = sol::make_layout(p.BH, p.Nq, p.Nk, p.d);
  const sol::WsPtrs ws = sol::make_ptrs(ws_base, lay);
  int n = 0;
  cudaError_t e = sol::launch_pool(p, static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k),
                                   static_cast<const __nv_bfloat16*>(v), ws, stream, &n);
  if (e == cudaSuccess && q) e = sol::launch_thresholds(p, ws, stream, &n);
  g_launches += n;
  return e == cudaSuccess ? SOL_OK : SOL_ERR_CUDA;
}

}  // namespace

namespace sol {
void count_launches(int n) { g_launches += n; }
sol_status_t check_device_arch() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SOL_ERR_CUDA;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return SOL_ERR_CUDA;
  return major == 10 ? SOL_OK : SOL_ERR_UNSUPPORTED_ARCH;
}
}  // namespace sol

extern "C" {

const char* sol_attn_status_string(sol_status_t s) {
  switch (s) {
    case SOL_OK: return "SOL_OK";
    case SOL_ERR_INVALID_ARG: return "SOL_ERR_INVALID_ARG";
    case SOL_ERR_UNSUPPORTED_SHAPE: return "SOL_ERR_UNSUPPORTED_SHAPE";
    case SOL_ERR_UNSUPPORTED_ARCH: return "SOL_ERR_UNSUPPORTED_ARCH";
    case SOL_ERR_WORKSPACE: return "SOL_ERR_WORKSPACE";
    case SOL_ERR_CUDA: return "SOL_ERR_CUDA";
    case SOL_ERR_DEVICE_TIMEOUT: return "SOL_ERR_DEVICE_TIMEOUT";
    case SOL_ERR_SCRATCH_LIMIT: return "SOL_ERR_SCRATCH_LIMIT";
    case SOL_ERR_STATIC_SCRATCH: return "SOL_ERR_STATIC_SCRATCH";
    default: return "SOL_ERR_UNKNOWN";
  }
}

size_t sol_attn_workspace_bytes(int B, int H, int N, int d, int block_q, int block_k) {
  if (check_shape(B, H, N, d, block_q, block_k, false) != SOL_OK) return 0;
  return sol::make_layout(B * H, sol::ceil_div(N, block_q), sol::ceil_div(N, block_k), d).total;
}

sol_status_t sol_attn_workspace_view(int B, int H, int N, int d, int block_q, int block_k, sol_attn_ws_view* view) {
  if (!view) return SOL_ERR_INVALID_ARG;
  sol_status_t s = check_shape(B, H, N, d, block_q, block_k, false);
  if (s != SOL_OK) return s;
  const int Nq = sol::ceil_div(N, block_q), Nk = sol::ceil_div(N, block_k);
  const sol::WsLayout w = sol::make_layout(B * H, Nq, Nk, d);
  view->status = w.status; view->qbar = w.qbar; view->kc = w.kc; view->vc = w.vc;
  view->mu = w.mu; view->sigma = w.sigma; view->tau = w.tau; view->total_bytes = w.total;
  view->n_q_blocks = Nq; view->n_k_blocks = Nk;
  return SOL_OK;
}

sol_status_t sol_attn_bind_workspace(void* dev_ws, size_t bytes, int32_t* dev_counts) {
  if (!dev_ws) { g_bound = Bound{}; return SOL_OK; }
  if ((reinterpret_cast<uintptr_t>(dev_ws) & 1023u) != 0) return SOL_ERR_WORKSPACE;
  if (bytes < 1024) return SOL_ERR_WORKSPACE;
  g_bound.ws = dev_ws; g_bound.bytes = bytes; g_bound.counts = dev_counts;
  return SOL_OK;
}

sol_status_t sol_attn_pool(const void* q, const void* k, const void* v, int B, int H, int N, int d,
                           int block_q, int block_k, float threshold, sol_stream_t stream) {
  sol_status_t s = check_shape(B, H, N, d, block_q, block_k, false);
  if (s != SOL_OK) return s;
  if (!k || !v || !aligned16(k) || !aligned16(v) || (q && !aligned16(q)) || std::isnan(threshold))
    return SOL_ERR_INVALID_ARG;
  if (!g_bound.ws) return SOL_ERR_WORKSPACE;
  if (g_bound.bytes < sol_attn_workspace_bytes(B, H, N, d, block_q, block_k)) return SOL_ERR_WORKSPACE;
  if ((s = check_arch()) != SOL_OK) return s;
  const sol::Problem p = make_problem(B, H, N, d, block_q, block_k, threshold, 0.f, SOL_MODE_SOL);
  return run_pool(p, q, k, v, g_bound.ws, static_cast<cudaStream_t>(stream));
}

sol_status_t sol_attn_thresholds(int B, int H, int N, int d, int block_q, int block_k, float threshold, float scale,
                                 int estimator, sol_stream_t stream) {
  sol_status_t s = check_shape(B, H, N, d, block_q, block_k, false);
  if (s != SOL_OK) return s;
  if (std::isnan(threshold) || std::isnan(scale) || std::isinf(scale)) return SOL_ERR_INVALID_ARG;
  if (estimator != SOL_EST_MOMENTS && estimator != SOL_EST_DIAGONAL) return SOL_ERR_INVALID_ARG;
  if (!g_bound.ws) return SOL_ERR_WORKSPACE;
  if (g_bound.bytes < sol_attn_workspace_bytes(B, H, N, d, block_q, block_k)) return SOL_ERR_WORKSPACE;
  if ((s = check_arch()) != SOL_OK) return s;
  const sol::Problem p = make_problem(B, H, N, d, block_q, block_k, threshold, scale, SOL_MODE_SOL, estimator);
  const sol::WsPtrs ws = sol::make_ptrs(g_bound.ws, sol::make_layout(p.BH, p.Nq, p.Nk, p.d));
  int n = 0;
  const cudaError_t e = sol::launch_thresholds(p, ws, static_cast<cudaStream_t>(stream), &n);
  g_launches += n;
  return e == cudaSuccess ? SOL_OK : SOL_ERR_CUDA;
}

sol_status_t sol_attn_route_mask(int B, int H, int N, int d, int block_q, int block_k, float scale,
                                 const float* tau_override, const uint8_t* forced_blocks, uint32_t* mask,
                                 sol_stream_t stream) {
  sol_status_t s = check_shape(B, H, N, d, block_q, block_k, false);
  if (s != SOL_OK) return s;
  if (!mask || std::isnan(scale) || std::isinf(scale)) return SOL_ERR_INVALID_ARG;
  if (!g_bound.ws) return SOL_ERR_WORKSPACE;
  if (g_bound.bytes < sol_attn_workspace_bytes(B, H, N, d, block_q, block_k)) return SOL_ERR_WORKSPACE;
  if ((s = check_arch()) != SOL_OK) return s;
  const sol::Problem p = make_problem(B, H, N, d, block_q, block_k, 0.f, scale, SOL_MODE_SOL, SOL_EST_MOMENTS,
                                      forced_blocks);
  const sol::WsPtrs ws = sol::make_ptrs(g_bound.ws, sol::make_layout(p.BH, p.Nq, p.Nk, p.d));
  int n = 0;
  const cudaError_t e = sol::launch_route_prepass(p, ws, tau_override ? tau_override : ws.tau, mask,
                                                  static_cast<cudaStream_t>(stream), &n);
  g_launches += n;
  return e == cudaSuccess ? SOL_OK : SOL_ERR_CUDA;
}

// keep_status: a later piece of one logical call must not wipe the device status of an earlier one
static sol_status_t forward_impl(const sol_attn_args* a, bool keep_status) {
  if (!a) return SOL_ERR_INVALID_ARG;
  sol_status_t s = check_shape(a->B, a->H, a->N, a->d, a->block_q, a->block_k, true);
  if (s != SOL_OK) return s;
  if (!a->q || !a->k || !a->v || !a->out) return SOL_ERR_INVALID_ARG;
  if (!aligned16(a->q) || !aligned16(a->k) || !aligned16(a->v) || !aligned16(a->out)) return SOL_ERR_INVALID_ARG;
  if (a->mode < SOL_MODE_SOL || a->mode > SOL_MODE_EXACT_ONLY) return SOL_ERR_INVALID_ARG;
  if (a->impl < SOL_IMPL_AUTO || a->impl > SOL_IMPL_MMA_SYNC) return SOL_ERR_INVALID_ARG;
  if (a->mode != SOL_MODE_DENSE && !a->tau_override && std::isnan(a->threshold)) return SOL_ERR_INVALID_ARG;
  if (std::isnan(a->scale) || std::isinf(a->scale)) return SOL_ERR_INVALID_ARG;
  if (a->estimator != SOL_EST_MOMENTS && a->estimator != SOL_EST_DIAGONAL) return SOL_ERR_INVALID_ARG;
  if (a->layout != SOL_LAYOUT_BHND && a->layout != SOL_LAYOUT_BNHD) return SOL_ERR_INVALID_ARG;
  if (a->routing != SOL_ROUTING_FUSED && a->routing != SOL_ROUTING_PREPASS) return SOL_ERR_INVALID_ARG;
  // the pre-pass keeps its decisions in the caller's mask buffer
  const bool prepass = a->routing == SOL_ROUTING_PREPASS && a->mode != SOL_MODE_DENSE;
  if (prepass && !a->mask_out) return SOL_ERR_INVALID_ARG;
  if (!a->workspace || (reinterpret_cast<uintptr_t>(a->workspace) & 1023u) != 0) return SOL_ERR_WORKSPACE;
  if (a->workspace_bytes < sol_attn_workspace_bytes(a->B, a->H, a->N, a->d, a->block_q, a->block_k))
    return SOL_ERR_WORKSPACE;
  if ((s = check_arch()) != SOL_OK) return s;

  sol::Problem p = make_problem(a->B, a->H, a->N, a->d, a->block_q, a->block_k, a->threshold, a->scale, a->mode,
                                a->estimator, a->mode == SOL_MODE_DENSE ? nullptr : a->forced_blocks, a->layout);
  p.routing = prepass ? SOL_ROUTING_PREPASS : SOL_ROUTING_FUSED;
  int impl = a->impl;
  if (impl == SOL_IMPL_AUTO) impl = sol::fwd_sm100_supports(p) ? SOL_IMPL_TCGEN05 : SOL_IMPL_MMA_SYNC;
  if (impl == SOL_IMPL_TCGEN05 && !sol::fwd_sm100_supports(p)) return SOL_ERR_UNSUPPORTED_SHAPE;
  if (prepass && impl != SOL_IMPL_TCGEN05) return SOL_ERR_INVALID_ARG;   // only the tcgen05 kernel reads the bits

  cudaStream_t stream = static_cast<cudaStream_t>(a->stream);
  const sol::WsLayout lay = sol::make_layout(p.BH, p.Nq, p.Nk, p.d);
  const sol::WsPtrs ws = sol::make_ptrs(a->workspace, lay);
  const int first_word = keep_status ? sol::kStatusTileCounter : 0;
  if (cudaMemsetAsync(ws.status + first_word, 0, sizeof(int32_t) * (sol::kStatusWords - first_word), stream) !=
      cudaSuccess)
    return SOL_ERR_CUDA;
  if (p.mode != SOL_MODE_DENSE && !a->skip_pool) {
    s = run_pool(p, a->q, a->k, a->v, a->workspace, stream);
    if (s != SOL_OK) return s;
  }
  const float* tau = a->tau_override ? a->tau_override : ws.tau;
  int n = 0;
  cudaError_t e;
  if (prepass) {
    e = sol::launch_route_prepass(p, ws, tau, a->mask_out, stream, &n);
    if (e != cudaSuccess) { g_launches += n; return SOL_ERR_CUDA; }
  }
  const auto* q = static_cast<const __nv_bfloat16*>(a->q);
  const auto* k = static_cast<const __nv_bfloat16*>(a->k);
  const auto* v = static_cast<const __nv_bfloat16*>(a->v);
  auto* out = static_cast<__nv_bfloat16*>(a->out);
  if (impl == SOL_IMPL_TCGEN05) e = sol::launch_fwd_sm100(p, q, k, v, out, ws, tau, a->counts, a->mask_out, stream, &n);
  else e = sol::launch_fwd_mma_sync(p, q, k, v, out, ws, tau, a->counts, a->mask_out, stream, &n);
  g_launches += n;
  return e == cudaSuccess ? SOL_OK : SOL_ERR_CUDA;
}

sol_status_t sol_attn_forward_ex(const sol_attn_args* a) { return forward_impl(a, false); }

sol_status_t sol_attn_forward(const void* q, const void* k, const void* v, void* out, int B, int H, int N,
                              int d, int block_q, int block_k, float threshold, sol_stream_t stream) {
  if (!g_bound.ws) return SOL_ERR_WORKSPACE;
  sol_attn_args a{};
  a.q = q; a.k = k; a.v = v; a.out = out;
  a.B = B; a.H = H; a.N = N; a.d = d; a.block_q = block_q; a.block_k = block_k;
  a.threshold = threshold; a.scale = 0.f; a.mode = SOL_MODE_SOL; a.impl = SOL_IMPL_AUTO;
  a.workspace = g_bound.ws; a.workspace_bytes = g_bound.bytes; a.counts = g_bound.counts;
  a.stream = stream;
  return sol_attn_forward_ex(&a);
}

sol_status_t sol_attn_dense(const void* q, const void* k, const void* v, void* out, int B, int H, int N,
                            int d, sol_stream_t stream) {
  if (!g_bound.ws) return SOL_ERR_WORKSPACE;
  sol_attn_args a{};
  a.q = q; a.k = k; a.v = v; a.out = out;
  a.B = B; a.H = H; a.N = N; a.d = d;
  a.block_q = a.block_k = (d == 64 ? 64 : 128);
  a.threshold = 0.f; a.scale = 0.f; a.mode = SOL_MODE_DENSE; a.impl = SOL_IMPL_AUTO;
  a.workspace = g_bound.ws; a.workspace_bytes = g_bound.bytes; a.counts = g_bound.counts;
  a.stream = stream;
  return sol_attn_forward_ex(&a);
}

sol_status_t sol_attn_forward_host(const void* hq, const void* hk, const void* hv, void* hout, void* dq, void* dk,
                                   void* dv, void* dout, int B, int H, int N, int d, int block_q, int block_k,
                                   float threshold, sol_stream_t stream) {
  if (!hq || !hk || !hv || !hout || !dq || !dk || !dv || !dout) return SOL_ERR_INVALID_ARG;
  sol_status_t s = check_shape(B, H, N, d, block_q, block_k, true);
  if (s != SOL_OK) return s;
  if (!g_bound.ws) return SOL_ERR_WORKSPACE;
  if (g_bound.bytes < sol_attn_workspace_bytes(B, H, N, d, block_q, block_k)) return SOL_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  HostPath hp;
  if ((s = host_path(&hp)) != SOL_OK) return s;

  // Heads are independent, so the call is cut into groups of heads and pipelined: while the
  // kernels work on one group (on the caller's stream), the next group's q, k, v travel to the
  // device on one copy stream and the previous group's output travels back on another.
  const int BH = B * H, Nq = sol::ceil_div(N, block_q);
  const size_t head_bytes = (size_t)N * d * 2;
  const size_t want = host_group_bytes();
  int per = (int)((want + head_bytes - 1) / head_bytes);
  if (per < 1) per = 1;
  if (per > BH) per = BH;
  // copies must not overtake work already queued on the caller's stream (it may still use dq...)
  if (cudaEventRecord(hp.start, st) != cudaSuccess || cudaStreamWaitEvent(hp.in, hp.start, 0) != cudaSuccess ||
      cudaStreamWaitEvent(hp.out, hp.start, 0) != cudaSuccess)
    return SOL_ERR_CUDA;
  bool first = true;
  for (int h0 = 0; h0 < BH; h0 += per) {
    const int nh = (BH - h0 < per) ? BH - h0 : per;
    const size_t off = (size_t)h0 * head_bytes, bytes = (size_t)nh * head_bytes;
    auto at = [off](const void* p) { return static_cast<const char*>(p) + off; };
    auto at_w = [off](void* p) { return static_cast<char*>(p) + off; };
    if (cudaMemcpyAsync(at_w(dq), at(hq), bytes, cudaMemcpyHostToDevice, hp.in) != cudaSuccess ||
        cudaMemcpyAsync(at_w(dk), at(hk), bytes, cudaMemcpyHostToDevice, hp.in) != cudaSuccess ||
        cudaMemcpyAsync(at_w(dv), at(hv), bytes, cudaMemcpyHostToDevice, hp.in) != cudaSuccess ||
        cudaEventRecord(hp.copied, hp.in) != cudaSuccess || cudaStreamWaitEvent(st, hp.copied, 0) != cudaSuccess)
      return SOL_ERR_CUDA;
    sol_attn_args a{};
    a.q = at_w(dq); a.k = at_w(dk); a.v = at_w(dv); a.out = at_w(dout);
    a.B = 1; a.H = nh; a.N = N; a.d = d; a.block_q = block_q; a.block_k = block_k;
    a.threshold = threshold; a.scale = 0.f; a.mode = SOL_MODE_SOL; a.impl = SOL_IMPL_AUTO;
    a.workspace = g_bound.ws; a.workspace_bytes = g_bound.bytes;
    a.counts = g_bound.counts ? g_bound.counts + (size_t)h0 * Nq : nullptr;
    a.stream = stream;
    s = forward_impl(&a, !first);
    first = false;
    if (s != SOL_OK) return s;
    if (cudaEventRecord(hp.computed, st) != cudaSuccess || cudaStreamWaitEvent(hp.out, hp.computed, 0) != cudaSuccess ||
        cudaMemcpyAsync(at_w(hout), at(dout), bytes, cudaMemcpyDeviceToHost, hp.out) != cudaSuccess)
      return SOL_ERR_CUDA;
  }
  // the caller's stream ends where the last copy back ends
  if (cudaEventRecord(hp.done, hp.out) != cudaSuccess || cudaStreamWaitEvent(st, hp.done, 0) != cudaSuccess)
    return SOL_ERR_CUDA;
  return SOL_OK;
}

sol_status_t sol_attn_read_device_status(sol_stream_t stream) {
  if (!g_bound.ws) return SOL_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t words[2] = {0, 0};
  if (cudaMemcpyAsync(words, g_bound.ws, sizeof(words), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SOL_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return SOL_ERR_CUDA;
  if (words[0] != 0) {
    cudaMemsetAsync(g_bound.ws, 0, sizeof(words), st);
    cudaStreamSynchronize(st);
    return static_cast<sol_status_t>(words[0]);
  }
  return SOL_OK;
}

int64_t sol_attn_launch_count(void) { return g_launches.load(); }

void sol_attn_debug_set_wait(int64_t wait_cycles, int32_t withhold_tile) {
  sol::fwd_sm100_set_wait(static_cast<long long>(wait_cycles), withhold_tile);
}

}  // extern "C"
