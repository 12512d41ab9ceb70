// Host side of libsgdb: argument checks, launch shapes and the C ABI declared in
// include/sgdb.h.  Nothing here allocates device memory, and no call synchronises
// the stream except sgdb_step_host, whose results are host buffers.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <limits>
#include <atomic>
#include <mutex>

#include "sgdb_kernels.cuh"

namespace {

using namespace sgdb;

constexpr int kVersion = 100;  // 0.1.0
constexpr int kMaxDevices = 64;

// Launch shape of the row-streaming kernel: 256 consumer threads + one producer warp,
// CH 16-byte chunks per thread and row, so a ring slot holds 8 KiB (f32) / 8 KiB (bf16).
#ifndef SGDB_NT
#define SGDB_NT 256
#endif
#ifndef SGDB_CH
#define SGDB_CH 2
#endif
#ifndef SGDB_CH_BF16
#define SGDB_CH_BF16 SGDB_CH
#endif
constexpr int kNT = SGDB_NT;
template <typename GT>
struct Shape {  // 16-byte chunks per thread and row, per gradient type
  static constexpr int kCH = SGDB_CH;
};
template <>
struct Shape<BF16> {
  static constexpr int kCH = SGDB_CH_BF16;
};
constexpr int kDefaultStages = 7;
constexpr int kDefaultCtasPerSm = 2;

struct DeviceInfo {
  std::atomic<bool> known{false};  // set last, with release: a reader that sees it sees the other fields
  int index = 0;
  int sms = 0;
  int max_smem_optin = 0;
};
DeviceInfo g_dev[kMaxDevices];
std::mutex g_dev_mutex;
std::atomic<long long> g_wait_limit_ns{static_cast<long long>(kWaitLimitNs)};
int g_stages = kDefaultStages;
int g_ctas_per_sm = kDefaultCtasPerSm;
constexpr int kDefaultArrivalBlocksPerSm = 4;
constexpr long long kDefaultArrivalResidentBytes = 96ll << 20;
int g_arrival_blocks_per_sm = kDefaultArrivalBlocksPerSm;
long long g_arrival_resident_bytes = kDefaultArrivalResidentBytes;

const float kNoDeadline = std::numeric_limits<float>::infinity();

bool is_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

sgdb_status_t device_info(const DeviceInfo** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SGDB_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return SGDB_ERR_UNSUPPORTED;
  DeviceInfo& d = g_dev[dev];
  if (!d.known.load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!d.known.load(std::memory_order_relaxed)) {
      if (cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
          cudaDeviceGetAttribute(&d.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) !=
              cudaSuccess)
        return SGDB_ERR_CUDA;
      d.index = dev;
      d.known.store(true, std::memory_order_release);
    }
  }
  *out = &d;
  return SGDB_OK;
}

sgdb_status_t launch_status() {
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    std::fprintf(stderr, "libsgdb: CUDA error: %s\n", cudaGetErrorString(e));
    return SGDB_ERR_CUDA;
  }
  return SGDB_OK;
}

bool dtype_ok(int dt) { return dt == SGDB_F32 || dt == SGDB_BF16; }
size_t dtype_size(int dt) { return dt == SGDB_BF16 ? 2 : 4; }

// Checks the optimizer description and the state pointers its rule needs; derives
// the constants the kernels use.  `ep` receives the epilogue selector.
sgdb_status_t prepare_rule(const sgdb_opt_t* opt, const void* state0, const void* state1, Hyper* h,
                           int* ep) {
  if (opt == nullptr) return SGDB_ERR_INVALID_ARG;
  std::memset(h, 0, sizeof(*h));
  if (!std::isfinite(opt->lr)) return SGDB_ERR_INVALID_ARG;
  h->lr = opt->lr;
  switch (opt->kind) {
    case SGDB_SGD:
      *ep = EP_SGD;
      return SGDB_OK;
    case SGDB_MOMENTUM:
      if (!std::isfinite(opt->momentum) || state0 == nullptr) return SGDB_ERR_INVALID_ARG;
      h->mu = opt->momentum;
      *ep = EP_MOMENTUM;
      return SGDB_OK;
    case SGDB_RMSPROP:
      if (!std::isfinite(opt->momentum) || !std::isfinite(opt->decay) || !std::isfinite(opt->eps) ||
          state0 == nullptr || state1 == nullptr)
        return SGDB_ERR_INVALID_ARG;
      h->mu = opt->momentum;
      h->rho = opt->decay;
      h->one_minus_rho = static_cast<float>(1.0 - static_cast<double>(opt->decay));
      h->eps = opt->eps;
      *ep = EP_RMSPROP;
      return SGDB_OK;
    case SGDB_ADAM: {
      if (!std::isfinite(opt->beta1) || !std::isfinite(opt->beta2) || !std::isfinite(opt->eps) ||
          opt->beta1 < 0.f || opt->beta1 >= 1.f || opt->beta2 < 0.f || opt->beta2 >= 1.f ||
          opt->step < 1 || state0 == nullptr || state1 == nullptr)
        return SGDB_ERR_INVALID_ARG;
      h->b1 = opt->beta1;
      h->b2 = opt->beta2;
      h->one_minus_b1 = static_cast<float>(1.0 - static_cast<double>(opt->beta1));
      h->one_minus_b2 = static_cast<float>(1.0 - static_cast<double>(opt->beta2));
      h->eps = opt->eps;
      const double k = static_cast<double>(opt->step);
      h->bc1 = static_cast<float>(1.0 - std::pow(static_cast<double>(opt->beta1), k));
      h->bc2 = static_cast<float>(1.0 - std::pow(static_cast<double>(opt->beta2), k));
      *ep = EP_ADAM;
      return SGDB_OK;
    }
    case SGDB_ADAGRAD:
      if (!std::isfinite(opt->eps) || state0 == nullptr) return SGDB_ERR_INVALID_ARG;
      h->eps = opt->eps;
      *ep = EP_ADAGRAD;
      return SGDB_OK;
    default:
      return SGDB_ERR_INVALID_ARG;
  }
}

sgdb_status_t check_selection_args(const void* arrival, const void* tags, int32_t N, int32_t b,
                                   const void* mask, const void* order, const void* info) {
  if (arrival == nullptr || tags == nullptr || mask == nullptr || order == nullptr || info == nullptr)
    return SGDB_ERR_INVALID_ARG;
  if (N < 1 || b < 0) return SGDB_ERR_INVALID_ARG;
  if (static_cast<int64_t>(N) + b > SGDB_MAX_WORKERS) return SGDB_ERR_INVALID_ARG;
  return SGDB_OK;
}

// ---------------------------------------------------------------- row-streaming launch

template <typename GT, int EP, bool GROUPED = false, bool ROWS = false>
sgdb_status_t launch_stream_t(const StreamParams& p_in, cudaStream_t stream) {
  const DeviceInfo* dev = nullptr;
  sgdb_status_t st = device_info(&dev);
  if (st != SGDB_OK) return st;
  StreamParams p = p_in;
  constexpr int kCH = Shape<GT>::kCH;
  constexpr int kStageBytes = kNT * kCH * 16;
  auto kernel = stream_rows_kernel<GT, EP, kNT, kCH, GROUPED, ROWS>;

  // shared memory: ring + 2 barriers per slot + order[N] + tile prefix[S + 1] + selection scratch
  if (p.order_cap < p.N) p.order_cap = p.N;
  const size_t fixed = static_cast<size_t>((p.order_cap + 3) & ~3) * 4 + (p.table ? (static_cast<size_t>(p.S) + 1) * 4 : 0) +
                       (p.arrival ? static_cast<size_t>(p.W) * 4 : 0) +
                       (GROUPED ? (4 * static_cast<size_t>(p.M) + static_cast<size_t>(p.N) + 1) * 4 : 0) +
                       (ROWS ? (static_cast<size_t>(p.order_cap) + static_cast<size_t>(p.R)) * 8 : 0) + 16;
  int ctas_per_sm = g_ctas_per_sm;
  int stages = g_stages;
  const size_t per_sm_budget = static_cast<size_t>(dev->max_smem_optin);
  // keep the requested residency: shrink the ring until `ctas_per_sm` blocks fit (1 KiB reserved per block)
  while (stages > 2 &&
         (static_cast<size_t>(stages) * (kStageBytes + 16) + fixed + 1024) * ctas_per_sm > per_sm_budget + 1024)
    --stages;
  const size_t smem = static_cast<size_t>(stages) * (kStageBytes + 16) + fixed;
  if (smem > per_sm_budget) return SGDB_ERR_UNSUPPORTED;
  p.stages = stages;
  p.wait_limit_ns = static_cast<unsigned long long>(g_wait_limit_ns.load(std::memory_order_relaxed));
  // the opt-in to large dynamic shared memory is kept per kernel and device: asked for again only when a
  // launch needs more than any launch of this kernel before it
  static std::atomic<int> smem_allowed[kMaxDevices];
  if (static_cast<int>(smem) > smem_allowed[dev->index].load(std::memory_order_relaxed)) {
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) !=
        cudaSuccess)
      return launch_status();
    smem_allowed[dev->index].store(static_cast<int>(smem), std::memory_order_relaxed);
  }
  long long grid = static_cast<long long>(dev->sms) * ctas_per_sm;
  if (p.table == nullptr) {
    const long long tile = static_cast<long long>(kNT) * kCH * GradTraits<GT>::kVec;
    p.total_tiles = static_cast<int>((p.flat.len + tile - 1) / tile);
    if (p.total_tiles < grid) grid = p.total_tiles;
  }
  if (grid < 1) grid = 1;
  kernel<<<static_cast<unsigned>(grid), kNT + 32, smem, stream>>>(p);
  return launch_status();
}

template <typename GT>
sgdb_status_t launch_stream_ep(int ep, const StreamParams& p, cudaStream_t stream) {
  switch (ep) {
    case EP_MEAN: return launch_stream_t<GT, EP_MEAN>(p, stream);
    case EP_SGD: return launch_stream_t<GT, EP_SGD>(p, stream);
    case EP_MOMENTUM: return launch_stream_t<GT, EP_MOMENTUM>(p, stream);
    case EP_RMSPROP: return launch_stream_t<GT, EP_RMSPROP>(p, stream);
    case EP_ADAM: return launch_stream_t<GT, EP_ADAM>(p, stream);
    case EP_ADAGRAD: return launch_stream_t<GT, EP_ADAGRAD>(p, stream);
  }
  return SGDB_ERR_INVALID_ARG;
}

sgdb_status_t launch_stream(int dt, int ep, const StreamParams& p, cudaStream_t stream) {
  return dt == SGDB_BF16 ? launch_stream_ep<BF16>(ep, p, stream) : launch_stream_ep<float>(ep, p, stream);
}

template <typename GT>
sgdb_status_t launch_stream_grouped_ep(int ep, const StreamParams& p, cudaStream_t stream) {
  switch (ep) {
    case EP_SGD: return launch_stream_t<GT, EP_SGD, true>(p, stream);
    case EP_MOMENTUM: return launch_stream_t<GT, EP_MOMENTUM, true>(p, stream);
    case EP_RMSPROP: return launch_stream_t<GT, EP_RMSPROP, true>(p, stream);
    case EP_ADAM: return launch_stream_t<GT, EP_ADAM, true>(p, stream);
    case EP_ADAGRAD: return launch_stream_t<GT, EP_ADAGRAD, true>(p, stream);
  }
  return SGDB_ERR_INVALID_ARG;
}

sgdb_status_t launch_stream_grouped(int dt, int ep, const StreamParams& p, cudaStream_t stream) {
  return dt == SGDB_BF16 ? launch_stream_grouped_ep<BF16>(ep, p, stream) : launch_stream_grouped_ep<float>(ep, p, stream);
}

template <typename GT>
sgdb_status_t launch_stream_rows_ep(int ep, const StreamParams& p, cudaStream_t stream) {
  switch (ep) {
    case EP_SGD: return launch_stream_t<GT, EP_SGD, false, true>(p, stream);
    case EP_MOMENTUM: return launch_stream_t<GT, EP_MOMENTUM, false, true>(p, stream);
    case EP_RMSPROP: return launch_stream_t<GT, EP_RMSPROP, false, true>(p, stream);
    case EP_ADAM: return launch_stream_t<GT, EP_ADAM, false, true>(p, stream);
    case EP_ADAGRAD: return launch_stream_t<GT, EP_ADAGRAD, false, true>(p, stream);
  }
  return SGDB_ERR_INVALID_ARG;
}

sgdb_status_t launch_stream_rows(int dt, int ep, const StreamParams& p, cudaStream_t stream) {
  return dt == SGDB_BF16 ? launch_stream_rows_ep<BF16>(ep, p, stream) : launch_stream_rows_ep<float>(ep, p, stream);
}

long long tiles_of(int dt, long long len) {
  const long long tile = dt == SGDB_BF16 ? static_cast<long long>(kNT) * Shape<BF16>::kCH * 8
                                         : static_cast<long long>(kNT) * Shape<float>::kCH * 4;
  return (len + tile - 1) / tile;
}

sgdb_status_t launch_select(const float* d_arrival, const int32_t* d_tags, int32_t t, int32_t N, int32_t b,
                            uint8_t* d_mask, int32_t* d_order, int32_t* d_info, cudaStream_t stream) {
  const int W = N + b;
  const int threads = (W + 31) & ~31;  // one thread per worker
  select_first_n_kernel<<<1, threads, 0, stream>>>(d_arrival, d_tags, t, N, W, kNoDeadline, false, d_mask, d_order,
                                                    d_info);
  return launch_status();
}

void set_in_kernel_selection(StreamParams* p, const float* d_arrival, const int32_t* d_tags, int32_t t, int32_t W,
                             uint8_t* d_mask, int32_t* d_order, int32_t* d_info) {
  p->order = nullptr;
  p->info = nullptr;
  p->status_out = d_info + 1;
  p->arrival = d_arrival;
  p->tags = d_tags;
  p->t = t;
  p->reverse = t & 1;  // consecutive iterations walk through the columns in opposite directions
  p->W = W;
  p->deadline = kNoDeadline;
  p->keep_all = false;
  p->order_cap = p->N;
  p->mask_out = d_mask;
  p->order_out = d_order;
  p->info_out = d_info;
}

// Parameters of the row-streaming kernel for one flat vector; selection fields are filled in by the caller.
StreamParams flat_params(float* theta, float* state0, float* state1, const void* grad, int64_t ld, int64_t P, int32_t N) {
  StreamParams p{};
  p.table = nullptr;
  p.flat.theta = theta;
  p.flat.state0 = state0;
  p.flat.state1 = state1;
  p.flat.grad = grad;
  p.flat.ld = ld;
  p.flat.len = P;
  p.S = 1;
  p.N = N;
  return p;
}

sgdb_status_t check_flat(const void* grad, int dt, int64_t P, int64_t ld, int32_t N) {
  if (grad == nullptr || !dtype_ok(dt)) return SGDB_ERR_INVALID_ARG;
  if (P < 0 || ld < P || N < 1 || N > SGDB_MAX_WORKERS) return SGDB_ERR_INVALID_ARG;
  if (!is_aligned16(grad)) return SGDB_ERR_INVALID_ARG;
  if (tiles_of(dt, P) > 0x7fffffffLL) return SGDB_ERR_UNSUPPORTED;
  return SGDB_OK;
}

// Launch with programmatic stream serialization, like every kernel that works on the server state.
template <typename Kernel, typename Params>
sgdb_status_t launch_on_server_state(Kernel kernel, unsigned grid, const Params& p, cudaStream_t s) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = SGDB_PDL ? 1 : 0;
  (void)cudaLaunchKernelEx(&cfg, kernel, p);
  return launch_status();
}

}  // namespace

// ====================================================================== C ABI

extern "C" {

sgdb_status_t sgdb_select(const float* d_arrival, const int32_t* d_tags, int32_t t, int32_t N, int32_t b,
                          uint8_t* d_mask, int32_t* d_order, int32_t* d_info, void* stream) {
  sgdb_status_t st = check_selection_args(d_arrival, d_tags, N, b, d_mask, d_order, d_info);
  if (st != SGDB_OK) return st;
  return launch_select(d_arrival, d_tags, t, N, b, d_mask, d_order, d_info, static_cast<cudaStream_t>(stream));
}

sgdb_status_t sgdb_aggregate(const void* d_grad, sgdb_dtype_t dt, int64_t P, int64_t ld, int32_t N,
                             const int32_t* d_order, const int32_t* d_info, float* d_mean, void* stream) {
  sgdb_status_t st = check_flat(d_grad, dt, P, ld, N);
  if (st != SGDB_OK) return st;
  if (d_order == nullptr || d_mean == nullptr || !is_aligned16(d_mean)) return SGDB_ERR_INVALID_ARG;
  if (P == 0) return SGDB_OK;
  StreamParams p = flat_params(d_mean, nullptr, nullptr, d_grad, ld, P, N);  // the mean goes where theta would
  p.order = d_order;
  p.info = d_info;
  return launch_stream(dt, EP_MEAN, p, static_cast<cudaStream_t>(stream));
}

sgdb_status_t sgdb_update(float* d_theta, float* d_state0, float* d_state1, const float* d_mean, int64_t P,
                          const sgdb_opt_t* opt, const int32_t* d_info, void* stream) {
  Hyper h;
  int ep = 0;
  sgdb_status_t st = prepare_rule(opt, d_state0, d_state1, &h, &ep);
  if (st != SGDB_OK) return st;
  if (d_theta == nullptr || d_mean == nullptr || P < 0) return SGDB_ERR_INVALID_ARG;
  if (!is_aligned16(d_theta) || !is_aligned16(d_mean) || !is_aligned16(d_state0) || !is_aligned16(d_state1))
    return SGDB_ERR_INVALID_ARG;
  if (P == 0) return SGDB_OK;
  const DeviceInfo* dev = nullptr;
  st = device_info(&dev);
  if (st != SGDB_OK) return st;
  UpdateParams p{d_theta, d_state0, d_state1, d_mean, P, d_info, h};
  const long long chunks = (P + 3) / 4;
  long long grid = (chunks + 2 * 256 - 1) / (2 * 256);  // two chunks per thread and pass
  const long long cap = static_cast<long long>(dev->sms) * 8;
  if (grid > cap) grid = cap;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  switch (ep) {
    case EP_SGD: update_kernel<EP_SGD><<<static_cast<unsigned>(grid), 256, 0, s>>>(p); break;
    case EP_MOMENTUM: update_kernel<EP_MOMENTUM><<<static_cast<unsigned>(grid), 256, 0, s>>>(p); break;
    case EP_RMSPROP: update_kernel<EP_RMSPROP><<<static_cast<unsigned>(grid), 256, 0, s>>>(p); break;
    case EP_ADAM: update_kernel<EP_ADAM><<<static_cast<unsigned>(grid), 256, 0, s>>>(p); break;
    case EP_ADAGRAD: update_kernel<EP_ADAGRAD><<<static_cast<unsigned>(grid), 256, 0, s>>>(p); break;
    default: return SGDB_ERR_INVALID_ARG;
  }
  return launch_status();
}

static sgdb_status_t step_flat(const void* d_grad, sgdb_dtype_t dt, int64_t P, int64_t ld, const float* d_arrival,
                               const int32_t* d_tags, int32_t t, int32_t N, int32_t b, float* d_theta,
                               float* d_state0, float* d_state1, const sgdb_opt_t* opt, uint8_t* d_mask,
                               int32_t* d_order, int32_t* d_info, float* d_ema, float alpha, void* stream) {
  sgdb_status_t st = check_selection_args(d_arrival, d_tags, N, b, d_mask, d_order, d_info);
  if (st != SGDB_OK) return st;
  st = check_flat(d_grad, dt, P, ld, N);
  if (st != SGDB_OK) return st;
  Hyper h;
  int ep = 0;
  st = prepare_rule(opt, d_state0, d_state1, &h, &ep);
  if (st != SGDB_OK) return st;
  if (d_theta == nullptr || !is_aligned16(d_theta) || !is_aligned16(d_state0) || !is_aligned16(d_state1) ||
      !is_aligned16(d_ema))
    return SGDB_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (P == 0) return launch_select(d_arrival, d_tags, t, N, b, d_mask, d_order, d_info, s);
  StreamParams p = flat_params(d_theta, d_state0, d_state1, d_grad, ld, P, N);
  set_in_kernel_selection(&p, d_arrival, d_tags, t, N + b, d_mask, d_order, d_info);
  p.ema = d_ema;
  p.ema_alpha = alpha;
  p.ema_one_minus_alpha = static_cast<float>(1.0 - static_cast<double>(alpha));
  p.h = h;
  return launch_stream(dt, ep, p, s);  // one launch: selection is the kernel's prologue
}

sgdb_status_t sgdb_step(const void* d_grad, sgdb_dtype_t dt, int64_t P, int64_t ld, const float* d_arrival,
                        const int32_t* d_tags, int32_t t, int32_t N, int32_t b, float* d_theta,
                        float* d_state0, float* d_state1, const sgdb_opt_t* opt, uint8_t* d_mask,
                        int32_t* d_order, int32_t* d_info, void* stream) {
  return step_flat(d_grad, dt, P, ld, d_arrival, d_tags, t, N, b, d_theta, d_state0, d_state1, opt, d_mask, d_order,
                   d_info, nullptr, 0.0f, stream);
}

sgdb_status_t sgdb_step_ema(const void* d_grad, sgdb_dtype_t dt, int64_t P, int64_t ld, const float* d_arrival,
                            const int32_t* d_tags, int32_t t, int32_t N, int32_t b, float* d_theta,
                            float* d_state0, float* d_state1, const sgdb_opt_t* opt, float* d_ema, float alpha,
                            uint8_t* d_mask, int32_t* d_order, int32_t* d_info, void* stream) {
  if (d_ema == nullptr || !(alpha >= 0.0f && alpha <= 1.0f)) return SGDB_ERR_INVALID_ARG;
  return step_flat(d_grad, dt, P, ld, d_arrival, d_tags, t, N, b, d_theta, d_state0, d_state1, opt, d_mask, d_order,
                   d_info, d_ema, alpha, stream);
}

sgdb_status_t sgdb_ema(float* d_ema, const float* d_theta, int64_t P, float alpha, const int32_t* d_info,
                       void* stream) {
  if (d_ema == nullptr || d_theta == nullptr || P < 0 || !(alpha >= 0.0f && alpha <= 1.0f)) return SGDB_ERR_INVALID_ARG;
  if (!is_aligned16(d_ema) || !is_aligned16(d_theta)) return SGDB_ERR_INVALID_ARG;
  if (P == 0) return SGDB_OK;
  const DeviceInfo* dev = nullptr;
  sgdb_status_t st = device_info(&dev);
  if (st != SGDB_OK) return st;
  EmaParams p{d_ema, d_theta, P, alpha, static_cast<float>(1.0 - static_cast<double>(alpha)), d_info};
  const long long chunks = (P + 3) / 4;
  long long grid = (chunks + 255) / 256;
  const long long cap = static_cast<long long>(dev->sms) * 8;
  if (grid > cap) grid = cap;
  ema_kernel<<<static_cast<unsigned>(grid), 256, 0, static_cast<cudaStream_t>(stream)>>>(p);
  return launch_status();
}

double sgdb_learning_rate(double gamma0, double beta, int64_t t, int64_t N, double T) {
  if (!(T > 0.0) || N < 1 || t < 0) return std::nan("");
  return gamma0 * std::pow(beta, static_cast<double>(t) * static_cast<double>(N) / (2.0 * T));
}

sgdb_status_t sgdb_select_deadline(const float* d_arrival, const int32_t* d_tags, int32_t t, int32_t W,
                                   float deadline, int32_t n_min, uint8_t* d_mask, int32_t* d_order,
                                   int32_t* d_info, void* stream) {
  if (W < 1 || n_min < 1 || n_min > W || std::isnan(deadline)) return SGDB_ERR_INVALID_ARG;
  sgdb_status_t st = check_selection_args(d_arrival, d_tags, W, 0, d_mask, d_order, d_info);
  if (st != SGDB_OK) return st;
  const int threads = (W + 31) & ~31;
  select_first_n_kernel<<<1, threads, 0, static_cast<cudaStream_t>(stream)>>>(d_arrival, d_tags, t, n_min, W, deadline,
                                                                              true, d_mask, d_order, d_info);
  return launch_status();
}

sgdb_status_t sgdb_step_deadline(const void* d_grad, sgdb_dtype_t dt, int64_t P, int64_t ld, const float* d_arrival,
                                 const int32_t* d_tags, int32_t t, int32_t W, float deadline, int32_t n_min,
                                 float* d_theta, float* d_state0, float* d_state1, const sgdb_opt_t* opt,
                                 uint8_t* d_mask, int32_t* d_order, int32_t* d_info, void* stream) {
  if (W < 1 || n_min < 1 || n_min > W || std::isnan(deadline)) return SGDB_ERR_INVALID_ARG;
  sgdb_status_t st = check_selection_args(d_arrival, d_tags, W, 0, d_mask, d_order, d_info);
  if (st != SGDB_OK) return st;
  st = check_flat(d_grad, dt, P, ld, n_min);
  if (st != SGDB_OK) return st;
  Hyper h;
  int ep = 0;
  st = prepare_rule(opt, d_state0, d_state1, &h, &ep);
  if (st != SGDB_OK) return st;
  if (d_theta == nullptr || !is_aligned16(d_theta) || !is_aligned16(d_state0) || !is_aligned16(d_state1))
    return SGDB_ERR_INVALID_ARG;
  if (P == 0) return sgdb_select_deadline(d_arrival, d_tags, t, W, deadline, n_min, d_mask, d_order, d_info, stream);
  StreamParams p = flat_params(d_theta, d_state0, d_state1, d_grad, ld, P, n_min);
  set_in_kernel_selection(&p, d_arrival, d_tags, t, W, d_mask, d_order, d_info);
  p.deadline = deadline;
  p.keep_all = true;
  p.order_cap = W;
  p.h = h;
  return launch_stream(dt, ep, p, static_cast<cudaStream_t>(stream));
}

// The multi-tensor step in its three forms: first-N rule, first-N rule with per-tensor averages, time-out rule.
static sgdb_status_t step_segmented(const sgdb_segment_t* d_segments, int32_t S, sgdb_dtype_t dt,
                                    const float* d_arrival, const int32_t* d_tags, int32_t t, int32_t N, int32_t b,
                                    bool keep_all, float deadline, const sgdb_opt_t* opt, float* const* d_ema,
                                    float alpha, uint8_t* d_mask, int32_t* d_order, int32_t* d_info, void* stream) {
  sgdb_status_t st = check_selection_args(d_arrival, d_tags, keep_all ? N + b : N, keep_all ? 0 : b, d_mask, d_order, d_info);
  if (st != SGDB_OK) return st;
  if (d_segments == nullptr || S < 0 || !dtype_ok(dt)) return SGDB_ERR_INVALID_ARG;
  if (S > SGDB_MAX_SEGMENTS) return SGDB_ERR_UNSUPPORTED;
  Hyper h;
  int ep = 0;
  // the table lives on the device; whether each segment carries the state pointers its
  // rule needs cannot be seen from here, so only the rule itself is checked
  const int dummy = 0;
  st = prepare_rule(opt, &dummy, &dummy, &h, &ep);
  if (st != SGDB_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int32_t W = N + b;
  if (S == 0) {
    if (!keep_all) return launch_select(d_arrival, d_tags, t, N, b, d_mask, d_order, d_info, s);
    return sgdb_select_deadline(d_arrival, d_tags, t, W, deadline, N, d_mask, d_order, d_info, stream);
  }
  StreamParams p{};
  p.table = d_segments;
  p.S = S;
  p.N = N;  // with the time-out rule: the fewest gradients accepted
  set_in_kernel_selection(&p, d_arrival, d_tags, t, W, d_mask, d_order, d_info);
  if (keep_all) {
    p.deadline = deadline;
    p.keep_all = true;
    p.order_cap = W;
  }
  p.ema_table = d_ema;
  p.ema_alpha = alpha;
  p.ema_one_minus_alpha = static_cast<float>(1.0 - static_cast<double>(alpha));
  p.h = h;
  return launch_stream(dt, ep, p, s);
}

sgdb_status_t sgdb_step_segmented(const sgdb_segment_t* d_segments, int32_t S, sgdb_dtype_t dt,
                                  const float* d_arrival, const int32_t* d_tags, int32_t t, int32_t N,
                                  int32_t b, const sgdb_opt_t* opt, uint8_t* d_mask, int32_t* d_order,
                                  int32_t* d_info, void* stream) {
  return step_segmented(d_segments, S, dt, d_arrival, d_tags, t, N, b, false, kNoDeadline, opt, nullptr, 0.0f, d_mask,
                        d_order, d_info, stream);
}

sgdb_status_t sgdb_step_segmented_ema(const sgdb_segment_t* d_segments, float* const* d_ema, float alpha, int32_t S,
                                      sgdb_dtype_t dt, const float* d_arrival, const int32_t* d_tags, int32_t t,
                                      int32_t N, int32_t b, const sgdb_opt_t* opt, uint8_t* d_mask, int32_t* d_order,
                                      int32_t* d_info, void* stream) {
  if (d_ema == nullptr || !(alpha >= 0.0f && alpha <= 1.0f)) return SGDB_ERR_INVALID_ARG;
  return step_segmented(d_segments, S, dt, d_arrival, d_tags, t, N, b, false, kNoDeadline, opt, d_ema, alpha, d_mask,
                        d_order, d_info, stream);
}

sgdb_status_t sgdb_step_segmented_deadline(const sgdb_segment_t* d_segments, int32_t S, sgdb_dtype_t dt,
                                           const float* d_arrival, const int32_t* d_tags, int32_t t, int32_t W,
                                           float deadline, int32_t n_min, const sgdb_opt_t* opt, uint8_t* d_mask,
                                           int32_t* d_order, int32_t* d_info, void* stream) {
  if (W < 1 || n_min < 1 || n_min > W || std::isnan(deadline)) return SGDB_ERR_INVALID_ARG;
  return step_segmented(d_segments, S, dt, d_arrival, d_tags, t, n_min, W - n_min, true, deadline, opt, nullptr, 0.0f,
                        d_mask, d_order, d_info, stream);
}

static sgdb_status_t check_grouped_args(const void* arrival, const void* tags, const void* group, int32_t W, int32_t M,
                                        int32_t N, const void* mask, const void* group_order, const void* order,
                                        const void* info) {
  if (arrival == nullptr || tags == nullptr || group == nullptr || mask == nullptr || group_order == nullptr ||
      order == nullptr || info == nullptr)
    return SGDB_ERR_INVALID_ARG;
  if (W < 1 || M < 1 || N < 1 || N > M) return SGDB_ERR_INVALID_ARG;
  if (W > SGDB_MAX_WORKERS || M > SGDB_MAX_WORKERS) return SGDB_ERR_INVALID_ARG;
  return SGDB_OK;
}

sgdb_status_t sgdb_select_grouped(const float* d_arrival, const int32_t* d_tags, const int32_t* d_group, int32_t t,
                                  int32_t W, int32_t M, int32_t N, uint8_t* d_mask, int32_t* d_group_order,
                                  int32_t* d_order, int32_t* d_info, void* stream) {
  sgdb_status_t st = check_grouped_args(d_arrival, d_tags, d_group, W, M, N, d_mask, d_group_order, d_order, d_info);
  if (st != SGDB_OK) return st;
  const int larger = W > M ? W : M;
  const int threads = (larger + 31) & ~31;
  select_grouped_kernel<<<1, threads, 0, static_cast<cudaStream_t>(stream)>>>(d_arrival, d_tags, d_group, t, N, W, M,
                                                                              d_mask, d_group_order, d_order, d_info);
  return launch_status();
}

sgdb_status_t sgdb_step_grouped(const void* d_grad, sgdb_dtype_t dt, int64_t P, int64_t ld, const float* d_arrival,
                                const int32_t* d_tags, const int32_t* d_group, int32_t t, int32_t W, int32_t M,
                                int32_t N, float* d_theta, float* d_state0, float* d_state1, const sgdb_opt_t* opt,
                                uint8_t* d_mask, int32_t* d_group_order, int32_t* d_order, int32_t* d_info,
                                void* stream) {
  sgdb_status_t st = check_grouped_args(d_arrival, d_tags, d_group, W, M, N, d_mask, d_group_order, d_order, d_info);
  if (st != SGDB_OK) return st;
  st = check_flat(d_grad, dt, P, ld, N);
  if (st != SGDB_OK) return st;
  Hyper h;
  int ep = 0;
  st = prepare_rule(opt, d_state0, d_state1, &h, &ep);
  if (st != SGDB_OK) return st;
  if (d_theta == nullptr || !is_aligned16(d_theta) || !is_aligned16(d_state0) || !is_aligned16(d_state1))
    return SGDB_ERR_INVALID_ARG;
  if (P == 0)
    return sgdb_select_grouped(d_arrival, d_tags, d_group, t, W, M, N, d_mask, d_group_order, d_order, d_info, stream);
  StreamParams p = flat_params(d_theta, d_state0, d_state1, d_grad, ld, P, N);
  set_in_kernel_selection(&p, d_arrival, d_tags, t, W, d_mask, d_order, d_info);
  p.order_cap = W;
  p.group = d_group;
  p.M = M;
  p.group_order_out = d_group_order;
  p.h = h;
  return launch_stream_grouped(dt, ep, p, static_cast<cudaStream_t>(stream));
}

// Checks and kernel parameters shared by the two forms of the step whose rows are given by address;
// the selection fields are filled in by the caller.  `ep` receives the epilogue selector.
static sgdb_status_t prepare_rows(const void* const* d_rows, int32_t W, sgdb_dtype_t dt, int64_t len, int32_t N,
                                  float* d_theta, float* d_state0, float* d_state1, const sgdb_opt_t* opt,
                                  float* const* d_replicas, int32_t R, StreamParams* p, int* ep) {
  if (d_rows == nullptr || !dtype_ok(dt) || len < 0 || N < 1 || W < N || W > SGDB_MAX_WORKERS) return SGDB_ERR_INVALID_ARG;
  if (R < 0 || R > SGDB_MAX_REPLICAS || (R > 0 && d_replicas == nullptr)) return SGDB_ERR_INVALID_ARG;
  if (tiles_of(dt, len) > 0x7fffffffLL) return SGDB_ERR_UNSUPPORTED;
  Hyper h;
  sgdb_status_t st = prepare_rule(opt, d_state0, d_state1, &h, ep);
  if (st != SGDB_OK) return st;
  if (d_theta == nullptr || !is_aligned16(d_theta) || !is_aligned16(d_state0) || !is_aligned16(d_state1))
    return SGDB_ERR_INVALID_ARG;
  *p = flat_params(d_theta, d_state0, d_state1, nullptr, 0, len, N);
  p->rows = d_rows;
  p->W_rows = W;
  p->replicas = d_replicas;
  p->R = R;
  p->h = h;
  p->order_cap = N;
  p->deadline = kNoDeadline;
  return SGDB_OK;
}

static sgdb_status_t arrival(const void* d_row, sgdb_dtype_t dt, int32_t row_tag, int32_t t, int32_t N, int64_t P,
                             float* d_acc, int32_t* d_counter, float* d_theta, float* d_state0, float* d_state1,
                             const sgdb_opt_t* opt, float* d_ema, float alpha, int32_t* d_info, void* stream) {
  if (d_row == nullptr || d_acc == nullptr || d_counter == nullptr || d_theta == nullptr || d_info == nullptr)
    return SGDB_ERR_INVALID_ARG;
  if (!dtype_ok(dt) || N < 1 || P < 0) return SGDB_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d_row) % dtype_size(dt) != 0) return SGDB_ERR_INVALID_ARG;
  if (!is_aligned16(d_acc) || !is_aligned16(d_theta) || !is_aligned16(d_state0) || !is_aligned16(d_state1) ||
      !is_aligned16(d_ema))
    return SGDB_ERR_INVALID_ARG;
  Hyper h;
  int ep = 0;
  sgdb_status_t st = prepare_rule(opt, d_state0, d_state1, &h, &ep);
  if (st != SGDB_OK) return st;
  const DeviceInfo* dev = nullptr;
  st = device_info(&dev);
  if (st != SGDB_OK) return st;
  ArrivalParams p{d_row, row_tag, t, N, P, d_acc, d_counter, d_theta, d_state0, d_state1, d_info,
                  d_ema, alpha, static_cast<float>(1.0 - static_cast<double>(alpha)), g_arrival_resident_bytes / 4, 1, h};
  const int V = dt == SGDB_BF16 ? 8 : 4;
  const long long chunks = (P + V - 1) / V;
  long long grid = (chunks + 4 * 256 - 1) / (4 * 256);  // at least 4 chunks per thread
  const long long cap = static_cast<long long>(dev->sms) * g_arrival_blocks_per_sm;
  if (grid > cap) grid = cap;
  if (row_tag != t || grid < 1) grid = 1;  // a wrongly tagged gradient only updates the bookkeeping
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const unsigned g = static_cast<unsigned>(grid);
#define SGDB_ARRIVAL_CASE(EPV)                                                                               \
  case EPV:                                                                                                  \
    return dt == SGDB_BF16 ? launch_on_server_state(accumulate_arrival_kernel<BF16, EPV>, g, p, s)           \
                           : launch_on_server_state(accumulate_arrival_kernel<float, EPV>, g, p, s);
  switch (ep) {
    SGDB_ARRIVAL_CASE(EP_SGD)
    SGDB_ARRIVAL_CASE(EP_MOMENTUM)
    SGDB_ARRIVAL_CASE(EP_RMSPROP)
    SGDB_ARRIVAL_CASE(EP_ADAM)
    SGDB_ARRIVAL_CASE(EP_ADAGRAD)
  }
#undef SGDB_ARRIVAL_CASE
  return SGDB_ERR_INVALID_ARG;
}

sgdb_status_t sgdb_accumulate_arrival(const void* d_row, sgdb_dtype_t dt, int32_t row_tag, int32_t t,
                                      int32_t N, int64_t P, float* d_acc, int32_t* d_counter,
                                      float* d_theta, float* d_state0, float* d_state1,
                                      const sgdb_opt_t* opt, int32_t* d_info, void* stream) {
  return arrival(d_row, dt, row_tag, t, N, P, d_acc, d_counter, d_theta, d_state0, d_state1, opt, nullptr, 0.0f, d_info,
                 stream);
}

sgdb_status_t sgdb_accumulate_arrival_ema(const void* d_row, sgdb_dtype_t dt, int32_t row_tag, int32_t t,
                                          int32_t N, int64_t P, float* d_acc, int32_t* d_counter,
                                          float* d_theta, float* d_state0, float* d_state1,
                                          const sgdb_opt_t* opt, float* d_ema, float alpha, int32_t* d_info,
                                          void* stream) {
  if (d_ema == nullptr || !(alpha >= 0.0f && alpha <= 1.0f)) return SGDB_ERR_INVALID_ARG;
  return arrival(d_row, dt, row_tag, t, N, P, d_acc, d_counter, d_theta, d_state0, d_state1, opt, d_ema, alpha, d_info,
                 stream);
}

sgdb_status_t sgdb_accumulate_arrival_deadline(const void* d_row, sgdb_dtype_t dt, int32_t row_tag, float row_arrival,
                                               int32_t t, float deadline, int64_t P, float* d_acc, int32_t* d_counter,
                                               int32_t* d_info, void* stream) {
  if (d_row == nullptr || d_acc == nullptr || d_counter == nullptr || d_info == nullptr) return SGDB_ERR_INVALID_ARG;
  if (!dtype_ok(dt) || P < 0 || std::isnan(deadline)) return SGDB_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d_row) % dtype_size(dt) != 0 || !is_aligned16(d_acc)) return SGDB_ERR_INVALID_ARG;
  const DeviceInfo* dev = nullptr;
  sgdb_status_t st = device_info(&dev);
  if (st != SGDB_OK) return st;
  const bool in_time = std::isfinite(row_arrival) && row_arrival <= deadline;
  // no upper count with the time-out rule: N is out of reach, so this launch never completes a set
  ArrivalParams p{d_row, row_tag, t, std::numeric_limits<int32_t>::max(), P, d_acc, d_counter, nullptr, nullptr, nullptr,
                  d_info, nullptr, 0.0f, 1.0f, g_arrival_resident_bytes / 4, in_time ? 1 : 0, Hyper{}};
  const int V = dt == SGDB_BF16 ? 8 : 4;
  const long long chunks = (P + V - 1) / V;
  long long grid = (chunks + 4 * 256 - 1) / (4 * 256);
  const long long cap = static_cast<long long>(dev->sms) * g_arrival_blocks_per_sm;
  if (grid > cap) grid = cap;
  if (row_tag != t || !in_time || grid < 1) grid = 1;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dt == SGDB_BF16) return launch_on_server_state(accumulate_arrival_kernel<BF16, EP_SGD>, static_cast<unsigned>(grid), p, s);
  return launch_on_server_state(accumulate_arrival_kernel<float, EP_SGD>, static_cast<unsigned>(grid), p, s);
}

sgdb_status_t sgdb_accumulate_close(int32_t t, int32_t n_min, int64_t P, const float* d_acc, int32_t* d_counter,
                                    float* d_theta, float* d_state0, float* d_state1, const sgdb_opt_t* opt,
                                    float* d_ema, float alpha, int32_t* d_info, void* stream) {
  if (d_acc == nullptr || d_counter == nullptr || d_theta == nullptr || d_info == nullptr) return SGDB_ERR_INVALID_ARG;
  if (n_min < 1 || P < 0) return SGDB_ERR_INVALID_ARG;
  if (d_ema != nullptr && !(alpha >= 0.0f && alpha <= 1.0f)) return SGDB_ERR_INVALID_ARG;
  if (!is_aligned16(d_acc) || !is_aligned16(d_theta) || !is_aligned16(d_state0) || !is_aligned16(d_state1) ||
      !is_aligned16(d_ema))
    return SGDB_ERR_INVALID_ARG;
  Hyper h;
  int ep = 0;
  sgdb_status_t st = prepare_rule(opt, d_state0, d_state1, &h, &ep);
  if (st != SGDB_OK) return st;
  const DeviceInfo* dev = nullptr;
  st = device_info(&dev);
  if (st != SGDB_OK) return st;
  CloseParams p{t, n_min, P, d_acc, d_counter, d_theta, d_state0, d_state1, d_info, d_ema, alpha,
                static_cast<float>(1.0 - static_cast<double>(alpha)), h};
  const long long chunks = (P + 3) / 4;
  long long grid = (chunks + 255) / 256;
  const long long cap = static_cast<long long>(dev->sms) * 8;
  if (grid > cap) grid = cap;
  if (grid < 1) grid = 1;
  const unsigned g = static_cast<unsigned>(grid);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  switch (ep) {
    case EP_SGD: return launch_on_server_state(close_iteration_kernel<EP_SGD>, g, p, s);
    case EP_MOMENTUM: return launch_on_server_state(close_iteration_kernel<EP_MOMENTUM>, g, p, s);
    case EP_RMSPROP: return launch_on_server_state(close_iteration_kernel<EP_RMSPROP>, g, p, s);
    case EP_ADAM: return launch_on_server_state(close_iteration_kernel<EP_ADAM>, g, p, s);
    case EP_ADAGRAD: return launch_on_server_state(close_iteration_kernel<EP_ADAGRAD>, g, p, s);
  }
  return SGDB_ERR_INVALID_ARG;
}

sgdb_status_t sgdb_step_rows(const void* const* d_rows, sgdb_dtype_t dt, int64_t len, const float* d_arrival,
                             const int32_t* d_tags, int32_t t, int32_t N, int32_t b, float* d_theta, float* d_state0,
                             float* d_state1, const sgdb_opt_t* opt, float* const* d_replicas, int32_t R,
                             uint8_t* d_mask, int32_t* d_order, int32_t* d_info, void* stream) {
  sgdb_status_t st = check_selection_args(d_arrival, d_tags, N, b, d_mask, d_order, d_info);
  if (st != SGDB_OK) return st;
  StreamParams p{};
  int ep = 0;
  st = prepare_rows(d_rows, N + b, dt, len, N, d_theta, d_state0, d_state1, opt, d_replicas, R, &p, &ep);
  if (st != SGDB_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (len == 0) return launch_select(d_arrival, d_tags, t, N, b, d_mask, d_order, d_info, s);
  set_in_kernel_selection(&p, d_arrival, d_tags, t, N + b, d_mask, d_order, d_info);
  return launch_stream_rows(dt, ep, p, s);
}

sgdb_status_t sgdb_step_rows_ordered(const void* const* d_rows, int32_t W, sgdb_dtype_t dt, int64_t len, int32_t N,
                                     const int32_t* d_order, int32_t* d_info, float* d_theta, float* d_state0,
                                     float* d_state1, const sgdb_opt_t* opt, float* const* d_replicas, int32_t R,
                                     void* stream) {
  if (d_order == nullptr || d_info == nullptr) return SGDB_ERR_INVALID_ARG;
  StreamParams p{};
  int ep = 0;
  sgdb_status_t st = prepare_rows(d_rows, W, dt, len, N, d_theta, d_state0, d_state1, opt, d_replicas, R, &p, &ep);
  if (st != SGDB_OK) return st;
  if (len == 0) return SGDB_OK;
  p.order = d_order;
  p.info = d_info;
  p.status_out = d_info + 1;
  return launch_stream_rows(dt, ep, p, static_cast<cudaStream_t>(stream));
}

sgdb_status_t sgdb_enable_peer_access(int32_t peer_device) {
  int dev = 0, count = 0, can = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceCount(&count) != cudaSuccess) return launch_status();
  if (peer_device < 0 || peer_device >= count) return SGDB_ERR_INVALID_ARG;
  if (peer_device == dev) return SGDB_OK;  // a device reaches its own memory as it is
  if (cudaDeviceCanAccessPeer(&can, dev, peer_device) != cudaSuccess) return launch_status();
  if (!can) return SGDB_ERR_UNSUPPORTED;
  const cudaError_t e = cudaDeviceEnablePeerAccess(peer_device, 0);
  if (e == cudaErrorPeerAccessAlreadyEnabled) {
    (void)cudaGetLastError();
    return SGDB_OK;
  }
  if (e != cudaSuccess) return launch_status();
  return SGDB_OK;
}

sgdb_status_t sgdb_shard_range(int64_t P, int32_t n_servers, int32_t j, int64_t* first, int64_t* len) {
  if (first == nullptr || len == nullptr || P < 0 || P > (INT64_MAX >> 1) || n_servers < 1 || j < 0 || j >= n_servers)
    return SGDB_ERR_INVALID_ARG;
  const int64_t a = SGDB_SHARD_ALIGN;
  const int64_t per = (P + n_servers - 1) / n_servers;
  const int64_t chunk = (per + a - 1) / a * a;
  const int64_t start = static_cast<int64_t>(j) * chunk;  // at most P + n_servers * (a + 1): no overflow
  const int64_t lo = start < P ? start : P;
  const int64_t rest = P - lo;
  *first = lo;
  *len = rest < chunk ? rest : chunk;
  return SGDB_OK;
}

// Workspace layout of sgdb_step_host: arrival[W] f32 | tags[W] i32 | order[N] i32 | info[2] i32 |
// mask[W] u8, rounded up to 256 bytes, then the gradient rows with a 16-byte-multiple pitch.
static size_t host_ws_header(int32_t N, int32_t b) {
  const size_t W = static_cast<size_t>(N) + b;
  const size_t raw = W * 4 + W * 4 + static_cast<size_t>(N) * 4 + 8 + W;
  return (raw + 255) & ~static_cast<size_t>(255);
}
static int64_t host_ws_pitch(sgdb_dtype_t dt, int64_t P) {
  const int64_t v = dt == SGDB_BF16 ? 8 : 4;
  return (P + v - 1) / v * v;
}

size_t sgdb_step_host_workspace_bytes(sgdb_dtype_t dt, int64_t P, int64_t ld, int32_t N, int32_t b) {
  if (!dtype_ok(dt) || P < 0 || ld < P || N < 1 || b < 0 || static_cast<int64_t>(N) + b > SGDB_MAX_WORKERS)
    return 0;
  return host_ws_header(N, b) +
         static_cast<size_t>(N + b) * static_cast<size_t>(host_ws_pitch(dt, P)) * dtype_size(dt);
}

sgdb_status_t sgdb_step_host(const void* h_grad, sgdb_dtype_t dt, int64_t P, int64_t ld, const float* h_arrival,
                             const int32_t* h_tags, int32_t t, int32_t N, int32_t b, float* d_theta,
                             float* d_state0, float* d_state1, const sgdb_opt_t* opt, float* h_theta_out,
                             uint8_t* h_mask, int32_t* h_order, int32_t* h_info, void* d_workspace,
                             size_t workspace_bytes, void* stream) {
  sgdb_status_t st = check_selection_args(h_arrival, h_tags, N, b, h_mask, h_order, h_info);
  if (st != SGDB_OK) return st;
  if (h_grad == nullptr || d_theta == nullptr || d_workspace == nullptr || !dtype_ok(dt) || P < 0 || ld < P)
    return SGDB_ERR_INVALID_ARG;
  if (!is_aligned16(d_workspace) || !is_aligned16(d_theta) || !is_aligned16(d_state0) || !is_aligned16(d_state1))
    return SGDB_ERR_INVALID_ARG;
  const size_t need = sgdb_step_host_workspace_bytes(dt, P, ld, N, b);
  if (need == 0 || workspace_bytes < need) return SGDB_ERR_INVALID_ARG;
  Hyper h;
  int ep = 0;
  st = prepare_rule(opt, d_state0, d_state1, &h, &ep);
  if (st != SGDB_OK) return st;

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t W = static_cast<size_t>(N) + b;
  unsigned char* ws = static_cast<unsigned char*>(d_workspace);
  float* d_arrival = reinterpret_cast<float*>(ws);
  int32_t* d_tags = reinterpret_cast<int32_t*>(ws + W * 4);
  int32_t* d_order = reinterpret_cast<int32_t*>(ws + W * 8);
  int32_t* d_info = d_order + N;
  uint8_t* d_mask = reinterpret_cast<uint8_t*>(d_info + 2);
  unsigned char* d_rows = ws + host_ws_header(N, b);
  const size_t esize = dtype_size(dt);
  const int64_t pitch = host_ws_pitch(dt, P);

  bool ok = cudaMemcpyAsync(d_arrival, h_arrival, W * 4, cudaMemcpyHostToDevice, s) == cudaSuccess &&
            cudaMemcpyAsync(d_tags, h_tags, W * 4, cudaMemcpyHostToDevice, s) == cudaSuccess;
  if (!ok) return launch_status();
  st = launch_select(d_arrival, d_tags, t, N, b, d_mask, d_order, d_info, s);
  if (st != SGDB_OK) return st;
  ok = cudaMemcpyAsync(h_info, d_info, 8, cudaMemcpyDeviceToHost, s) == cudaSuccess &&
       cudaStreamSynchronize(s) == cudaSuccess;
  if (!ok) return launch_status();
  if (h_info[1] != SGDB_OK) return static_cast<sgdb_status_t>(h_info[1]);
  ok = cudaMemcpyAsync(h_order, d_order, static_cast<size_t>(N) * 4, cudaMemcpyDeviceToHost, s) == cudaSuccess &&
       cudaMemcpyAsync(h_mask, d_mask, W, cudaMemcpyDeviceToHost, s) == cudaSuccess &&
       cudaStreamSynchronize(s) == cudaSuccess;
  if (!ok) return launch_status();

  if (P > 0) {
    // only the kept rows cross to the device, each to the slot of its worker id
    for (int32_t k = 0; k < N; ++k) {
      const size_t w = static_cast<size_t>(h_order[k]);
      if (cudaMemcpyAsync(d_rows + w * static_cast<size_t>(pitch) * esize,
                          static_cast<const unsigned char*>(h_grad) + w * static_cast<size_t>(ld) * esize,
                          static_cast<size_t>(P) * esize, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return launch_status();
    }
    StreamParams p = flat_params(d_theta, d_state0, d_state1, d_rows, pitch, P, N);
    p.order = d_order;
    p.info = d_info;
    p.status_out = d_info + 1;
    p.reverse = t & 1;
    p.h = h;
    st = launch_stream(dt, ep, p, s);
    if (st != SGDB_OK) return st;
    if (h_theta_out != nullptr &&
        cudaMemcpyAsync(h_theta_out, d_theta, static_cast<size_t>(P) * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess)
      return launch_status();
    if (cudaMemcpyAsync(h_info, d_info, 8, cudaMemcpyDeviceToHost, s) != cudaSuccess) return launch_status();
  }
  if (cudaStreamSynchronize(s) != cudaSuccess) return launch_status();
  return static_cast<sgdb_status_t>(h_info[1]);
}

// ---------------------------------------------------------------- fixed-scratch variant
//
// Scratch for callers that cannot allocate: a file-scope device array.  In host code
// the name `g_static_scratch` is only a handle for the runtime, not a device address;
// the address each device gave the array is looked up once per device with
// cudaGetSymbolAddress (that device current) and it is that pointer the kernels get.
static __device__ __align__(256) unsigned char g_static_scratch[SGDB_STATIC_SCRATCH_BYTES];
static void* g_static_scratch_addr[kMaxDevices];  // per device, null until looked up
static std::mutex g_static_scratch_mutex;

sgdb_status_t sgdb_step_host_static(const void* h_grad, sgdb_dtype_t dt, int64_t P, int64_t ld,
                                    const float* h_arrival, const int32_t* h_tags, int32_t t, int32_t N,
                                    int32_t b, float* d_theta, float* d_state0, float* d_state1,
                                    const sgdb_opt_t* opt, float* h_theta_out, uint8_t* h_mask,
                                    int32_t* h_order, int32_t* h_info, void* stream) {
  const size_t need = sgdb_step_host_workspace_bytes(dt, P, ld, N, b);
  if (need == 0) return SGDB_ERR_INVALID_ARG;
  if (need > SGDB_STATIC_SCRATCH_BYTES) {
    std::fprintf(stderr,
                 "libsgdb: sgdb_step_host_static needs %zu bytes of scratch for these sizes, the built-in "
                 "array holds %u; use sgdb_step_host with a caller-owned workspace\n",
                 need, static_cast<unsigned>(SGDB_STATIC_SCRATCH_BYTES));
    return SGDB_ERR_UNSUPPORTED;
  }
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return launch_status();
  if (dev < 0 || dev >= kMaxDevices) return SGDB_ERR_UNSUPPORTED;
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (g_static_scratch_addr[dev] == nullptr) {
      void* addr = nullptr;
      const cudaError_t e = cudaGetSymbolAddress(&addr, g_static_scratch);
      if (e != cudaSuccess || addr == nullptr) {
        std::fprintf(stderr, "libsgdb: cudaGetSymbolAddress failed on device %d: %s\n", dev, cudaGetErrorString(e));
        (void)cudaGetLastError();
        return SGDB_ERR_CUDA;
      }
      g_static_scratch_addr[dev] = addr;
    }
    scratch = g_static_scratch_addr[dev];
  }
  return sgdb_step_host(h_grad, dt, P, ld, h_arrival, h_tags, t, N, b, d_theta, d_state0, d_state1, opt,
                        h_theta_out, h_mask, h_order, h_info, scratch, SGDB_STATIC_SCRATCH_BYTES, stream);
}

sgdb_status_t sgdb_set_tuning(int32_t stages, int32_t ctas_per_sm) {
  if (stages > 64 || ctas_per_sm > 8) return SGDB_ERR_INVALID_ARG;
  g_stages = stages > 0 ? (stages < 2 ? 2 : stages) : kDefaultStages;
  g_ctas_per_sm = ctas_per_sm > 0 ? ctas_per_sm : kDefaultCtasPerSm;
  return SGDB_OK;
}

sgdb_status_t sgdb_set_wait_limit_ns(int64_t limit_ns) {
  if (limit_ns > 10ll * 1000 * 1000 * 1000) return SGDB_ERR_INVALID_ARG;
  g_wait_limit_ns.store(limit_ns >= 0 ? limit_ns : static_cast<long long>(kWaitLimitNs), std::memory_order_relaxed);
  return SGDB_OK;
}

sgdb_status_t sgdb_set_arrival_tuning(int64_t resident_bytes, int32_t blocks_per_sm) {
  if (blocks_per_sm > 8) return SGDB_ERR_INVALID_ARG;
  g_arrival_resident_bytes = resident_bytes >= 0 ? resident_bytes : kDefaultArrivalResidentBytes;
  g_arrival_blocks_per_sm = blocks_per_sm > 0 ? blocks_per_sm : kDefaultArrivalBlocksPerSm;
  return SGDB_OK;
}

sgdb_status_t sgdb_selftest_bounded_wait(int64_t limit_ns, int32_t* d_out, void* stream) {
  if (d_out == nullptr || limit_ns < 0 || limit_ns > 100ll * 1000 * 1000) return SGDB_ERR_INVALID_ARG;
  bounded_wait_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<unsigned long long>(limit_ns),
                                                                                d_out);
  return launch_status();
}

const char* sgdb_strerror(sgdb_status_t status) {
  switch (status) {
    case SGDB_OK: return "ok";
    case SGDB_ERR_INVALID_ARG: return "invalid argument";
    case SGDB_ERR_INSUFFICIENT: return "fewer than N gradients carry the current iteration tag";
    case SGDB_ERR_CUDA: return "CUDA runtime or launch error";
    case SGDB_ERR_UNSUPPORTED: return "unsupported size or configuration";
    case SGDB_ERR_TIMEOUT: return "a bounded on-chip wait ran out";
  }
  return "unknown status";
}

int sgdb_version(void) { return kVersion; }

}  // extern "C"
