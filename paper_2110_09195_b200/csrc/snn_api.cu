// Host side of the C ABI declared in include/snn_conv.h: argument checks,
// the layer handle, path selection and the launches.  No arithmetic of the
// method happens on the host.
#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <tuple>
#include <utility>

#include "snn_internal.h"

using namespace snn;

namespace {

thread_local char g_err[512] = "";
std::atomic<long long> g_launches{0};

snn_status_t fail(snn_status_t st, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  if (getenv("SNN_LOG")) fprintf(stderr, "[snnconv] error %d: %s\n", (int)st, g_err);
  return st;
}

snn_status_t cuda_fail(cudaError_t e, const char* what) {
  snn_status_t st = (e == cudaErrorMemoryAllocation) ? SNN_ERR_OOM : SNN_ERR_CUDA;
  return fail(st, "%s: %s", what, cudaGetErrorString(e));
}

struct DeviceGuard {
  int prev = -1;
  bool ok = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) return;
    ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    int cur = -1;
    if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

}  // namespace

struct snn_conv {
  int C, K, tau, stride, pad, act_type, device;
  int ksize = 3;
  LayerDev L;
  std::mutex mu;
  std::map<std::tuple<int, int, int>, int> tuned;        // (N,H,W) -> path measured fastest by snn_conv_tune
  // (N,H,W, packed-sign output?) -> tensor-core plan and weight operand (a group of one)
  std::map<std::tuple<int, int, int, int>, GroupDev*> solo;
  // staging for snn_conv_forward_host
  void* stage_in = nullptr;
  void* stage_out = nullptr;
  size_t stage_in_bytes = 0, stage_out_bytes = 0;
  cudaStream_t host_stream = nullptr;
  int* tc_status_host = nullptr;  // pinned, written by the tensor-core kernel on a bounded-wait timeout
  int* tc_status_dev = nullptr;   // the same word as the device sees it
};

namespace {

bool make_geom(const snn_conv* h, int N, int H, int W, Geom* g) {
  if (N < 0 || H < 1 || W < 1) return false;
  if (H + 2 * h->pad < h->ksize || W + 2 * h->pad < h->ksize) return false;
  g->N = N; g->H = H; g->W = W;
  g->C = h->C; g->K = h->K; g->Cw = (h->C + 31) / 32;
  g->stride = h->stride; g->pad = h->pad;
  g->Ho = (H + 2 * h->pad - h->ksize) / h->stride + 1;
  g->Wo = (W + 2 * h->pad - h->ksize) / h->stride + 1;
  g->tau = h->tau; g->T = 1 << h->tau;
  g->ksize = h->ksize;
  // index arithmetic in the kernels is 32-bit for pixel counts
  long long in_px = (long long)N * H * W, out_px = (long long)N * g->Ho * g->Wo;
  if (in_px >= (1ll << 31) || out_px >= (1ll << 31)) return false;
  return true;
}

bool path_ok(const snn_conv* h, int path, const Geom& g) {
  switch (path) {
    case SNN_PATH_REUSE: return g.ksize == 3 && reuse_supported(g, h->act_type);
    case SNN_PATH_DECODED: return g.ksize == 3 && popc_supported(g, h->act_type);
    case SNN_PATH_DECODED_TC: return tcg_supported(g, h->act_type);
    default: return false;
  }
}

// Untuned default: tensor cores when they apply, else the popcount path for
// small c_out relative to the codebook and the reuse path for large (Sec. 4.5:
// sharing pays in proportion to c_out / 2^tau).  0 when no path can run the layer.
int heuristic_path(const snn_conv* h, const Geom& g) {
  if (path_ok(h, SNN_PATH_DECODED_TC, g)) return SNN_PATH_DECODED_TC;
  if (h->act_type == SNN_ACT_BIN) {
    if (g.K >= 4 * g.T && path_ok(h, SNN_PATH_REUSE, g)) return SNN_PATH_REUSE;
    if (path_ok(h, SNN_PATH_DECODED, g)) return SNN_PATH_DECODED;
  }
  if (path_ok(h, SNN_PATH_REUSE, g)) return SNN_PATH_REUSE;
  return 0;
}

int auto_path(snn_conv* h, const Geom& g) {
  if (const char* f = getenv("SNN_FORCE_PATH")) {
    int v = atoi(f);
    if (v >= 1 && v <= 3 && path_ok(h, v, g)) return v;
  }
  {
    std::lock_guard<std::mutex> lk(h->mu);
    auto it = h->tuned.find(std::make_tuple(g.N, g.H, g.W));
    if (it != h->tuned.end()) return it->second;
  }
  return heuristic_path(h, g);
}

// The tensor-core kernel's plan and weight operand for this input shape: built (and allocated) at the first
// call for the shape, reused afterwards.
cudaError_t solo_group(snn_conv* h, const Geom& g, int out_type, GroupDev** out, int* launched) {
  std::lock_guard<std::mutex> lk(h->mu);
  const int kind = out_type == SNN_OUT_BITS ? TCG_SIGNS : TCG_WORDS;
  const auto key = std::make_tuple(g.N, g.H, g.W, kind);
  auto it = h->solo.find(key);
  if (it != h->solo.end()) { *out = it->second; return cudaSuccess; }
  const LayerDev* Lp = &h->L;
  GroupDev* G = nullptr;
  cudaError_t e = tcg_create(&Lp, &g, 1, h->act_type, kind, h->host_stream, &G, launched);
  if (e != cudaSuccess) return e;
  h->solo[key] = G;
  *out = G;
  return cudaSuccess;
}

snn_status_t run_path(snn_conv* h, int path, const Geom& g, const Launch& l) {
  int launched = 0;
  cudaError_t e = cudaSuccess;
  switch (path) {
    case SNN_PATH_REUSE: e = reuse_forward(h->L, g, h->act_type, l, &launched); break;
    case SNN_PATH_DECODED: e = popc_forward(h->L, g, l, &launched); break;
    case SNN_PATH_DECODED_TC: {
      GroupDev* G = nullptr;
      e = solo_group(h, g, l.out_i32, &G, &launched);
      if (e == cudaSuccess) e = tcg_forward(G, &l.act, &l.out, l.out_i32, l.stream, h->tc_status_dev, &launched);
      break;
    }
    default: return fail(SNN_ERR_INVALID_ARG, "unknown path %d", path);
  }
  g_launches += launched;
  if (e != cudaSuccess) return cuda_fail(e, "kernel launch");
  return SNN_OK;
}

snn_status_t check_forward_args(snn_conv* h, const void* act, int N, int H, int W, void* out, int out_type, int path,
                                Geom* g, int* chosen) {
  if (!h) return fail(SNN_ERR_INVALID_ARG, "null handle");
  if (out_type != SNN_OUT_F32 && out_type != SNN_OUT_I32 && out_type != SNN_OUT_BITS)
    return fail(SNN_ERR_INVALID_ARG, "bad out_type %d", out_type);
  if (out_type != SNN_OUT_F32 && h->act_type != SNN_ACT_BIN)
    return fail(SNN_ERR_INVALID_ARG, "int32 and packed-sign outputs need binary activations");
  if (path < SNN_PATH_AUTO || path > SNN_PATH_DECODED_TC) return fail(SNN_ERR_INVALID_ARG, "unknown path %d", path);
  if (!make_geom(h, N, H, W, g))
    return fail(SNN_ERR_INVALID_ARG, "shape N=%d H=%d W=%d gives no output (pad %d) or is too large", N, H, W, h->pad);
  if (N > 0 && (!act || !out)) return fail(SNN_ERR_INVALID_ARG, "null activation / output pointer");
  if (((uintptr_t)act & 15) || ((uintptr_t)out & 15))
    return fail(SNN_ERR_INVALID_ARG, "activation / output pointers must be 16-byte aligned");
  int pth = path;
  if (out_type == SNN_OUT_BITS) {
    // only the tensor-core path writes packed signs
    if (pth != SNN_PATH_AUTO && pth != SNN_PATH_DECODED_TC)
      return fail(SNN_ERR_UNSUPPORTED, "packed-sign output is written by the tensor-core path only, not by path %d", pth);
    pth = SNN_PATH_DECODED_TC;
    if (!path_ok(h, pth, *g))
      return fail(SNN_ERR_UNSUPPORTED, "packed-sign output needs the tensor-core path, which cannot run this layer");
  } else if (pth == SNN_PATH_AUTO) {
    pth = auto_path(h, *g);
    if (pth < SNN_PATH_REUSE || !path_ok(h, pth, *g))
      return fail(SNN_ERR_UNSUPPORTED, "no path can run this layer at this shape (act_type %d, C=%d K=%d, N=%d %dx%d)",
                  h->act_type, h->C, h->K, N, H, W);
  } else if (!path_ok(h, pth, *g))
    return fail(SNN_ERR_UNSUPPORTED, "path %d does not support this layer (act_type %d, C=%d K=%d)", pth, h->act_type,
                h->C, h->K);
  *chosen = pth;
  return SNN_OK;
}

size_t act_bytes(const snn_conv* h, const Geom& g) {
  size_t px = (size_t)g.N * g.H * g.W;
  return h->act_type == SNN_ACT_BIN ? px * g.Cw * 4 : px * g.C * 2;
}
size_t out_bytes(const Geom& g) { return (size_t)g.N * g.Ho * g.Wo * g.K * 4; }

}  // namespace

namespace snn {
// used by snn_static.cu
snn_status_t api_fail(snn_status_t st, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  if (getenv("SNN_LOG")) fprintf(stderr, "[snnconv] error %d: %s\n", (int)st, g_err);
  return st;
}
void api_count_launches(int n) { g_launches += n; }
}  // namespace snn

extern "C" {

const char* snn_last_error(void) { return g_err; }
const char* snn_version(void) { return "snnconv 0.1 (sm_100a)"; }
int64_t snn_kernel_launches(void) { return (int64_t)g_launches.load(); }

snn_status_t snn_conv_create(const snn_conv_desc_t* d, snn_conv_t** out) {
  if (!out) return fail(SNN_ERR_INVALID_ARG, "null out pointer");
  *out = nullptr;
  if (!d) return fail(SNN_ERR_INVALID_ARG, "null descriptor");
  if (!d->codebook || !d->idx_packed || !d->alpha) return fail(SNN_ERR_INVALID_ARG, "null codebook / index / alpha");
  if (d->c_in < 1 || d->c_out < 1) return fail(SNN_ERR_INVALID_ARG, "c_in=%d c_out=%d", d->c_in, d->c_out);
  if (d->c_in > (1 << 16) || d->c_out > (1 << 16)) return fail(SNN_ERR_INVALID_ARG, "channel count above 65536");
  if (d->ksize != 0 && d->ksize != 1 && d->ksize != 3) return fail(SNN_ERR_INVALID_ARG, "ksize=%d is not 1 or 3", d->ksize);
  const bool one = d->ksize == 1;
  if (d->tau < 1 || d->tau > (one ? 8 : 9)) return fail(SNN_ERR_INVALID_ARG, "tau=%d outside 1..%d", d->tau, one ? 8 : 9);
  if (one && (d->c_in % 8)) return fail(SNN_ERR_INVALID_ARG, "a 1x1 layer needs c_in divisible by 8, not %d", d->c_in);
  if (one && d->pad != 0) return fail(SNN_ERR_INVALID_ARG, "a 1x1 layer takes no padding");
  if (d->stride < 1 || d->stride > 2) return fail(SNN_ERR_INVALID_ARG, "stride=%d outside {1,2}", d->stride);
  if (d->pad < 0 || d->pad > 1) return fail(SNN_ERR_INVALID_ARG, "pad=%d outside {0,1}", d->pad);
  if (d->act_type != SNN_ACT_BIN && d->act_type != SNN_ACT_F16)
    return fail(SNN_ERR_INVALID_ARG, "act_type=%d", d->act_type);
  const int T = 1 << d->tau;
  for (int j = 0; j < T; ++j)
    if (d->codebook[j] >= (one ? 256 : 512))
      return fail(SNN_ERR_INVALID_ARG, "codebook[%d]=%u is not a %d-bit code", j, d->codebook[j], one ? 8 : 9);
  for (int k = 0; k < d->c_out; ++k)
    if (!std::isfinite(d->alpha[k])) return fail(SNN_ERR_INVALID_ARG, "alpha[%d] is not finite", k);
  for (int k = 0; d->shift && k < d->c_out; ++k)
    if (!std::isfinite(d->shift[k])) return fail(SNN_ERR_INVALID_ARG, "shift[%d] is not finite", k);
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
    cudaGetLastError();
    return fail(SNN_ERR_CUDA, "no CUDA device available (this library has no CPU path)");
  }
  if (d->device < 0 || d->device >= ndev) return fail(SNN_ERR_INVALID_ARG, "device %d of %d", d->device, ndev);
  DeviceGuard guard(d->device);
  if (!guard.ok) return fail(SNN_ERR_CUDA, "cannot select device %d", d->device);

  snn_conv* h = new (std::nothrow) snn_conv();
  if (!h) return fail(SNN_ERR_OOM, "host allocation failed");
  h->C = d->c_in; h->K = d->c_out; h->tau = d->tau; h->stride = d->stride; h->pad = d->pad;
  h->act_type = d->act_type; h->device = d->device;
  h->ksize = one ? 1 : 3;
  Geom g;
  make_geom(h, 0, 3, 3, &g);
  const size_t n_elem = (size_t)h->K * (one ? h->C / 8 : h->C);
  const size_t idx_bytes = (n_elem * h->tau + 7) / 8;
  const int Tp = (T + 15) / 16 * 16;
  uint8_t* d_stream = nullptr;
  cudaError_t e = cudaSuccess;
  auto alloc = [&](void** p, size_t bytes) {
    if (e == cudaSuccess) e = cudaMalloc(p, bytes ? bytes : 16);
  };
  alloc((void**)&d_stream, idx_bytes + 4);
  alloc((void**)&h->L.idx, n_elem * 2);
  alloc((void**)&h->L.codebook, (size_t)T * 2);
  alloc((void**)&h->L.alpha, (size_t)h->K * 4);
  alloc((void**)&h->L.shift, (size_t)h->K * 4);
  alloc((void**)&h->L.wplanes, (size_t)9 * g.Cw * h->K * 4);
  alloc((void**)&h->L.corr, (size_t)16 * h->K * 4);
  alloc((void**)&h->L.match9, (size_t)Tp * 512);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->host_stream, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaHostAlloc((void**)&h->tc_status_host, sizeof(int), cudaHostAllocMapped);
  if (e == cudaSuccess) *h->tc_status_host = 0;
  if (e == cudaSuccess) e = cudaHostGetDevicePointer((void**)&h->tc_status_dev, h->tc_status_host, 0);
  cudaStream_t s = h->host_stream;
  if (e == cudaSuccess) e = cudaMemcpyAsync(d_stream, d->idx_packed, idx_bytes, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(h->L.codebook, d->codebook, (size_t)T * 2, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(h->L.alpha, d->alpha, (size_t)h->K * 4, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess)
    e = d->shift ? cudaMemcpyAsync(h->L.shift, d->shift, (size_t)h->K * 4, cudaMemcpyHostToDevice, s)
                 : cudaMemsetAsync(h->L.shift, 0, (size_t)h->K * 4, s);
  int launched = 0;
  if (e == cudaSuccess) e = decode_layer(h->L, d_stream, g, h->act_type, s, &launched);
  g_launches += launched;
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (d_stream) cudaFree(d_stream);
  if (e != cudaSuccess) {
    snn_status_t st = cuda_fail(e, "snn_conv_create");
    snn_conv_destroy(h);
    cudaGetLastError();
    return st;
  }
  *out = h;
  return SNN_OK;
}

snn_status_t snn_conv_destroy(snn_conv_t* h) {
  if (!h) return SNN_OK;
  DeviceGuard guard(h->device);
  cudaFree(h->L.idx);
  cudaFree(h->L.codebook);
  cudaFree(h->L.alpha);
  cudaFree(h->L.shift);
  cudaFree(h->L.wplanes);
  cudaFree(h->L.corr);
  cudaFree(h->L.match9);
  for (auto& kv : h->solo) tcg_destroy(kv.second);
  cudaFree(h->stage_in);
  cudaFree(h->stage_out);
  if (h->tc_status_host) cudaFreeHost(h->tc_status_host);
  if (h->host_stream) cudaStreamDestroy(h->host_stream);
  delete h;
  return SNN_OK;
}

snn_status_t snn_conv_forward(snn_conv_t* h, const void* act_dev, int32_t N, int32_t H, int32_t W, void* out_dev,
                              int32_t out_type, int32_t path, void* cuda_stream) {
  Geom g;
  int chosen = 0;
  snn_status_t st = check_forward_args(h, act_dev, N, H, W, out_dev, out_type, path, &g, &chosen);
  if (st != SNN_OK) return st;
  if (N == 0) return SNN_OK;
  DeviceGuard guard(h->device);
  if (!guard.ok) return fail(SNN_ERR_CUDA, "cannot select device %d", h->device);
  if (h->tc_status_host && *h->tc_status_host) {
    int code = *h->tc_status_host;
    *h->tc_status_host = 0;
    return fail(SNN_ERR_TIMEOUT, "an earlier tensor-core launch gave up a bounded wait (code %d)", code);
  }
  Launch l{act_dev, out_dev, out_type, (cudaStream_t)cuda_stream};
  return run_path(h, chosen, g, l);
}

snn_status_t snn_conv_forward_host(snn_conv_t* h, const void* act_host, int32_t N, int32_t H, int32_t W,
                                   void* out_host, int32_t out_type, int32_t path) {
  if (!h) return fail(SNN_ERR_INVALID_ARG, "null handle");
  Geom g;
  if (!make_geom(h, N, H, W, &g)) return fail(SNN_ERR_INVALID_ARG, "shape N=%d H=%d W=%d gives no output", N, H, W);
  if (N == 0) return SNN_OK;
  if (!act_host || !out_host) return fail(SNN_ERR_INVALID_ARG, "null host pointer");
  DeviceGuard guard(h->device);
  if (!guard.ok) return fail(SNN_ERR_CUDA, "cannot select device %d", h->device);
  const size_t ib = act_bytes(h, g);
  const size_t ob = out_type == SNN_OUT_BITS ? (size_t)g.N * g.Ho * g.Wo * ((g.K + 31) / 32) * 4 : out_bytes(g);
  cudaError_t e = cudaSuccess;
  if (ib > h->stage_in_bytes) {
    cudaFree(h->stage_in);
    h->stage_in = nullptr; h->stage_in_bytes = 0;
    e = cudaMalloc(&h->stage_in, ib);
    if (e != cudaSuccess) return cuda_fail(e, "staging input");
    h->stage_in_bytes = ib;
  }
  if (ob > h->stage_out_bytes) {
    cudaFree(h->stage_out);
    h->stage_out = nullptr; h->stage_out_bytes = 0;
    e = cudaMalloc(&h->stage_out, ob);
    if (e != cudaSuccess) return cuda_fail(e, "staging output");
    h->stage_out_bytes = ob;
  }
  cudaStream_t s = h->host_stream;
  e = cudaMemcpyAsync(h->stage_in, act_host, ib, cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return cuda_fail(e, "host to device copy");
  snn_status_t st = snn_conv_forward(h, h->stage_in, N, H, W, h->stage_out, out_type, path, (void*)s);
  if (st != SNN_OK) return st;
  e = cudaMemcpyAsync(out_host, h->stage_out, ob, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_fail(e, "device to host copy");
  if (h->tc_status_host && *h->tc_status_host) {
    int code = *h->tc_status_host;
    *h->tc_status_host = 0;
    return fail(SNN_ERR_TIMEOUT, "tensor-core kernel gave up a bounded wait (code %d)", code);
  }
  return SNN_OK;
}

snn_status_t snn_conv_path_supported(const snn_conv_t* h, int32_t path, int32_t N, int32_t H, int32_t W) {
  if (!h) return fail(SNN_ERR_INVALID_ARG, "null handle");
  Geom g;
  if (!make_geom(h, N, H, W, &g)) return fail(SNN_ERR_INVALID_ARG, "shape gives no output");
  if (path == SNN_PATH_AUTO) return SNN_OK;
  return path_ok(h, path, g) ? SNN_OK : SNN_ERR_UNSUPPORTED;
}

int32_t snn_conv_chosen_path(const snn_conv_t* h, int32_t N, int32_t H, int32_t W) {
  if (!h) return SNN_PATH_AUTO;
  Geom g;
  if (!make_geom(h, N, H, W, &g)) return SNN_PATH_AUTO;
  return auto_path(const_cast<snn_conv*>(h), g);
}

snn_status_t snn_conv_tune(snn_conv_t* h, int32_t N, int32_t H, int32_t W, int32_t* best_path, float* ms) {
  if (!h) return fail(SNN_ERR_INVALID_ARG, "null handle");
  Geom g;
  if (!make_geom(h, N, H, W, &g) || N < 1) return fail(SNN_ERR_INVALID_ARG, "shape gives no output");
  DeviceGuard guard(h->device);
  if (!guard.ok) return fail(SNN_ERR_CUDA, "cannot select device %d", h->device);
  void *a = nullptr, *o = nullptr;
  cudaError_t e = cudaMalloc(&a, act_bytes(h, g));
  if (e == cudaSuccess) e = cudaMalloc(&o, out_bytes(g));
  if (e == cudaSuccess) e = cudaMemset(a, 0x5a, act_bytes(h, g));
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  if (e == cudaSuccess) e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  if (e != cudaSuccess) {
    cudaFree(a); cudaFree(o);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    return cuda_fail(e, "snn_conv_tune setup");
  }
  if (h->act_type == SNN_ACT_BIN && (h->C & 31)) {
    // keep the unused high bits of the last word zero, as the layout requires
    // (0x5a5a5a5a has bits above C set): clear and use an all -1 input instead
    cudaMemset(a, 0, act_bytes(h, g));
  }
  if (h->act_type == SNN_ACT_F16) cudaMemset(a, 0x3c, act_bytes(h, g));  // 0x3c3c = 1.0586 in fp16
  cudaStream_t s = h->host_stream;
  float best = -1.f;
  int best_p = 0;
  snn_status_t st = SNN_OK;
  auto time_one = [&](int pth, float* t_out) -> snn_status_t {
    Launch l{a, o, 0, s};
    const int reps = 5;
    snn_status_t r = SNN_OK;
    for (int w = 0; w < 2 && r == SNN_OK; ++w) r = run_path(h, pth, g, l);
    if (r != SNN_OK) return r;
    cudaEventRecord(e0, s);
    for (int k = 0; k < reps && r == SNN_OK; ++k) r = run_path(h, pth, g, l);
    cudaEventRecord(e1, s);
    cudaError_t ce = cudaEventSynchronize(e1);
    if (r != SNN_OK) return r;
    if (ce != cudaSuccess) return cuda_fail(ce, "snn_conv_tune timing");
    float t = 0.f;
    cudaEventElapsedTime(&t, e0, e1);
    *t_out = t / reps;
    return SNN_OK;
  };
  for (int pth = 1; pth <= 3 && st == SNN_OK; ++pth) {
    if (ms) ms[pth] = -1.f;
    if (!path_ok(h, pth, g)) continue;
    float t = 0.f;
    st = time_one(pth, &t);
    if (st != SNN_OK) break;
    if (ms) ms[pth] = t;
    if (best < 0.f || t < best) { best = t; best_p = pth; }
  }
  if (ms) ms[0] = best;
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  cudaFree(a);
  cudaFree(o);
  if (st != SNN_OK) return st;
  if (!best_p) return fail(SNN_ERR_UNSUPPORTED, "no path supports this layer");
  {
    std::lock_guard<std::mutex> lk(h->mu);
    h->tuned[std::make_tuple(N, H, W)] = best_p;
  }
  if (best_path) *best_path = best_p;
  if (getenv("SNN_LOG"))
    fprintf(stderr, "[snnconv] tuned C=%d K=%d tau=%d N=%d %dx%d -> path %d (%.4f ms)\n", h->C, h->K, h->tau, N, H, W,
            best_p, best);
  return SNN_OK;
}

struct snn_conv_group {
  int device = 0, count = 0, act_type = 0;
  GroupDev* G = nullptr;        // planned for fp32 / int32 outputs
  GroupDev* G_signs = nullptr;  // planned for packed-sign outputs (binary activations only)
  int* status_host = nullptr;  // pinned, written by the kernel on a bounded-wait timeout
  int* status_dev = nullptr;
};

snn_status_t snn_conv_group_create(snn_conv_t* const* layers, int32_t count, const int32_t* N, const int32_t* H,
                                   const int32_t* W, snn_conv_group_t** out) {
  if (!out) return fail(SNN_ERR_INVALID_ARG, "null output pointer");
  *out = nullptr;
  if (!layers || !N || !H || !W) return fail(SNN_ERR_INVALID_ARG, "null argument");
  if (count < 1 || count > SNN_GROUP_MAX)
    return fail(SNN_ERR_INVALID_ARG, "a group has 1..%d members, not %d", SNN_GROUP_MAX, count);
  const LayerDev* Ls[SNN_GROUP_MAX];
  Geom gs[SNN_GROUP_MAX];
  for (int i = 0; i < count; ++i) {
    if (!layers[i]) return fail(SNN_ERR_INVALID_ARG, "member %d is a null handle", i);
    if (layers[i]->act_type != layers[0]->act_type || layers[i]->device != layers[0]->device)
      return fail(SNN_ERR_INVALID_ARG, "member %d differs from member 0 in activation type or device", i);
    if (N[i] < 1 || !make_geom(layers[i], N[i], H[i], W[i], &gs[i]))
      return fail(SNN_ERR_INVALID_ARG, "member %d: shape N=%d H=%d W=%d gives no output", i, N[i], H[i], W[i]);
    Ls[i] = &layers[i]->L;
  }
  DeviceGuard guard(layers[0]->device);
  if (!guard.ok) return fail(SNN_ERR_CUDA, "cannot select device %d", layers[0]->device);
  snn_conv_group* g = new (std::nothrow) snn_conv_group();
  if (!g) return fail(SNN_ERR_OOM, "host allocation failed");
  g->device = layers[0]->device;
  g->count = count;
  g->act_type = layers[0]->act_type;
  cudaError_t e = cudaHostAlloc((void**)&g->status_host, sizeof(int), cudaHostAllocMapped);
  if (e == cudaSuccess) {
    *g->status_host = 0;
    e = cudaHostGetDevicePointer((void**)&g->status_dev, g->status_host, 0);
  }
  int launched = 0;
  if (e == cudaSuccess) e = tcg_create(Ls, gs, count, g->act_type, TCG_WORDS, layers[0]->host_stream, &g->G, &launched);
  if (e == cudaSuccess && g->act_type == SNN_ACT_BIN)
    e = tcg_create(Ls, gs, count, g->act_type, TCG_SIGNS, layers[0]->host_stream, &g->G_signs, &launched);
  g_launches += launched;
  if (e != cudaSuccess) {
    tcg_destroy(g->G);
    tcg_destroy(g->G_signs);
    if (g->status_host) cudaFreeHost(g->status_host);
    delete g;
    if (e == cudaErrorInvalidConfiguration) {
      cudaGetLastError();
      return fail(SNN_ERR_UNSUPPORTED, "the grouped tensor-core kernel cannot run one of these layers at this shape");
    }
    return cuda_fail(e, "snn_conv_group_create");
  }
  *out = g;
  return SNN_OK;
}

snn_status_t snn_conv_group_forward(snn_conv_group_t* g, const void* const* act_dev, void* const* out_dev,
                                    int32_t out_type, void* cuda_stream) {
  if (!g || !g->G) return fail(SNN_ERR_INVALID_ARG, "null group");
  if (!act_dev || !out_dev) return fail(SNN_ERR_INVALID_ARG, "null pointer array");
  if (out_type != SNN_OUT_F32 && out_type != SNN_OUT_I32 && out_type != SNN_OUT_BITS)
    return fail(SNN_ERR_INVALID_ARG, "unknown output type %d", out_type);
  if (out_type != SNN_OUT_F32 && g->act_type != SNN_ACT_BIN)
    return fail(SNN_ERR_INVALID_ARG, "int32 and packed-sign outputs need binary activations");
  for (int i = 0; i < g->count; ++i) {
    if (!act_dev[i] || !out_dev[i]) return fail(SNN_ERR_INVALID_ARG, "member %d: null device pointer", i);
    if (((uintptr_t)act_dev[i] & 15) || ((uintptr_t)out_dev[i] & 15))
      return fail(SNN_ERR_INVALID_ARG, "member %d: misaligned device pointer", i);
  }
  DeviceGuard guard(g->device);
  if (!guard.ok) return fail(SNN_ERR_CUDA, "cannot select device %d", g->device);
  if (*g->status_host) {
    const int code = *g->status_host;
    *g->status_host = 0;
    return fail(SNN_ERR_TIMEOUT, "an earlier launch of the group gave up a bounded wait (code %d)", code);
  }
  int launched = 0;
  cudaError_t e = tcg_forward(out_type == SNN_OUT_BITS ? g->G_signs : g->G, act_dev, out_dev, out_type,
                              (cudaStream_t)cuda_stream, g->status_dev, &launched);
  g_launches += launched;
  if (e != cudaSuccess) return cuda_fail(e, "snn_conv_group_forward");
  return SNN_OK;
}

snn_status_t snn_conv_group_destroy(snn_conv_group_t* g) {
  if (!g) return SNN_OK;
  DeviceGuard guard(g->device);
  tcg_destroy(g->G);
  tcg_destroy(g->G_signs);
  if (g->status_host) cudaFreeHost(g->status_host);
  delete g;
  return SNN_OK;
}

struct snn_conv_stack {
  int device = 0, count = 0;
  GroupDev* G = nullptr;
  int* status_host = nullptr;  // pinned, written by the kernel on a bounded-wait timeout
  int* status_dev = nullptr;
};

snn_status_t snn_conv_stack_create(snn_conv_t* const* layers, int32_t count, int32_t N, int32_t H, int32_t W,
                                   snn_conv_stack_t** out) {
  if (!out) return fail(SNN_ERR_INVALID_ARG, "null output pointer");
  *out = nullptr;
  if (!layers) return fail(SNN_ERR_INVALID_ARG, "null argument");
  if (count < 1 || count > SNN_GROUP_MAX)
    return fail(SNN_ERR_INVALID_ARG, "a stack has 1..%d members, not %d", SNN_GROUP_MAX, count);
  const LayerDev* Ls[SNN_GROUP_MAX];
  Geom gs[SNN_GROUP_MAX];
  int h_in = H, w_in = W;
  for (int i = 0; i < count; ++i) {
    if (!layers[i]) return fail(SNN_ERR_INVALID_ARG, "member %d is a null handle", i);
    if (layers[i]->act_type != SNN_ACT_BIN)
      return fail(SNN_ERR_INVALID_ARG, "member %d: a stack chains binary activations", i);
    if (layers[i]->device != layers[0]->device) return fail(SNN_ERR_INVALID_ARG, "member %d is on another device", i);
    if (i > 0 && layers[i]->C != layers[i - 1]->K)
      return fail(SNN_ERR_INVALID_ARG, "member %d takes %d channels, member %d gives %d", i, layers[i]->C, i - 1,
                  layers[i - 1]->K);
    if (N < 1 || !make_geom(layers[i], N, h_in, w_in, &gs[i]))
      return fail(SNN_ERR_INVALID_ARG, "member %d: shape N=%d H=%d W=%d gives no output", i, N, h_in, w_in);
    if (!tcg_supported(gs[i], SNN_ACT_BIN))
      return fail(SNN_ERR_UNSUPPORTED, "member %d: the tensor-core path cannot run this layer at this shape", i);
    h_in = gs[i].Ho;
    w_in = gs[i].Wo;
    Ls[i] = &layers[i]->L;
  }
  DeviceGuard guard(layers[0]->device);
  if (!guard.ok) return fail(SNN_ERR_CUDA, "cannot select device %d", layers[0]->device);
  snn_conv_stack* st = new (std::nothrow) snn_conv_stack();
  if (!st) return fail(SNN_ERR_OOM, "host allocation failed");
  st->device = layers[0]->device;
  st->count = count;
  cudaError_t e = cudaHostAlloc((void**)&st->status_host, sizeof(int), cudaHostAllocMapped);
  if (e == cudaSuccess) {
    *st->status_host = 0;
    e = cudaHostGetDevicePointer((void**)&st->status_dev, st->status_host, 0);
  }
  int launched = 0;
  if (e == cudaSuccess) e = tcg_create(Ls, gs, count, SNN_ACT_BIN, TCG_CHAIN, layers[0]->host_stream, &st->G, &launched);
  g_launches += launched;
  if (e != cudaSuccess) {
    if (st->status_host) cudaFreeHost(st->status_host);
    delete st;
    if (e == cudaErrorInvalidConfiguration) {
      cudaGetLastError();
      return fail(SNN_ERR_UNSUPPORTED, "the tensor-core kernel cannot run these layers as one stack");
    }
    return cuda_fail(e, "snn_conv_stack_create");
  }
  *out = st;
  return SNN_OK;
}

snn_status_t snn_conv_stack_forward(snn_conv_stack_t* st, const void* act_dev, void* out_dev, int32_t out_type,
                                    void* cuda_stream) {
  if (!st || !st->G) return fail(SNN_ERR_INVALID_ARG, "null stack");
  if (!act_dev || !out_dev) return fail(SNN_ERR_INVALID_ARG, "null device pointer");
  if (out_type != SNN_OUT_F32 && out_type != SNN_OUT_I32 && out_type != SNN_OUT_BITS)
    return fail(SNN_ERR_INVALID_ARG, "unknown output type %d", out_type);
  if (((uintptr_t)act_dev & 15) || ((uintptr_t)out_dev & 15)) return fail(SNN_ERR_INVALID_ARG, "misaligned device pointer");
  DeviceGuard guard(st->device);
  if (!guard.ok) return fail(SNN_ERR_CUDA, "cannot select device %d", st->device);
  if (*st->status_host) {
    const int code = *st->status_host;
    *st->status_host = 0;
    return fail(SNN_ERR_TIMEOUT, "an earlier launch of the stack gave up a bounded wait (code %d)", code);
  }
  int launched = 0;
  cudaError_t e = tcg_forward(st->G, &act_dev, &out_dev, out_type, (cudaStream_t)cuda_stream, st->status_dev, &launched);
  g_launches += launched;
  if (e != cudaSuccess) return cuda_fail(e, "snn_conv_stack_forward");
  return SNN_OK;
}

snn_status_t snn_conv_stack_destroy(snn_conv_stack_t* st) {
  if (!st) return SNN_OK;
  DeviceGuard guard(st->device);
  tcg_destroy(st->G);
  if (st->status_host) cudaFreeHost(st->status_host);
  delete st;
  return SNN_OK;
}

snn_status_t snn_microbench(int32_t kind, int32_t device, double* rate) {
  if (!rate) return fail(SNN_ERR_INVALID_ARG, "null rate pointer");
  if (kind < 0 || kind > 9) return fail(SNN_ERR_INVALID_ARG, "unknown microbenchmark %d", kind);
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
    cudaGetLastError();
    return fail(SNN_ERR_CUDA, "device %d not available", device);
  }
  DeviceGuard guard(device);
  if (!guard.ok) return fail(SNN_ERR_CUDA, "cannot select device %d", device);
  cudaError_t e = microbench(kind, rate);
  g_launches += 2;
  if (kind == 9) {
    // self-test of the bounded waits: giving up is the expected outcome
    if (e == cudaErrorTimeout) return fail(SNN_ERR_TIMEOUT, "self-test: the wait gave up after %.3f s and reported it", *rate);
    if (e == cudaSuccess) return fail(SNN_ERR_CUDA, "self-test: a wait on a barrier nothing arrives on came back without a report");
  }
  if (e != cudaSuccess) return cuda_fail(e, "snn_microbench");
  return SNN_OK;
}

}  // extern "C"
