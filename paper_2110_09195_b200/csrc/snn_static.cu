// snn_conv_forward_static: the forward pass for callers that may not allocate.
//
// Everything the ordinary path keeps in buffers it allocates at create time
// (the copied index stream, unpacked indices, codebook, scales, decoded weight
// bit-planes, border corrections) lives here in ONE fixed device array that is
// part of the library image.  Each call copies the layer description into that
// array, decodes it there and runs the XOR + popcount kernel on it.
#include <cmath>
#include <cstdio>
#include <mutex>

#include "snn_internal.h"

using namespace snn;

namespace {

constexpr size_t kStaticScratchBytes = SNN_STATIC_SCRATCH_BYTES;

// The scratch itself.  Every GPU that loads the library holds these bytes until
// the process exits.  In host code this name is only a handle for the runtime,
// never a device address: the address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mu;
unsigned char* g_scratch_dev[kMaxDevices] = {nullptr};

// Device address of the scratch on the current device, resolved once per device.
cudaError_t scratch_address(int device, unsigned char** out) {
  std::lock_guard<std::mutex> lk(g_setup_mu);
  if (!g_scratch_dev[device]) {
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_dev[device] = static_cast<unsigned char*>(ptr);
  }
  *out = g_scratch_dev[device];
  return cudaSuccess;
}

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace

namespace snn {
// defined in snn_api.cu
snn_status_t api_fail(snn_status_t st, const char* fmt, ...);
void api_count_launches(int n);
}  // namespace snn

extern "C" SNN_API snn_status_t snn_conv_forward_static(const snn_conv_desc_t* d, const void* act_dev, int32_t N,
                                                        int32_t H, int32_t W, void* out_dev, int32_t out_type,
                                                        void* cuda_stream) {
  if (!d) return api_fail(SNN_ERR_INVALID_ARG, "null descriptor");
  if (!d->codebook || !d->idx_packed || !d->alpha) return api_fail(SNN_ERR_INVALID_ARG, "null codebook / index / alpha");
  if (d->c_in < 1 || d->c_out < 1) return api_fail(SNN_ERR_INVALID_ARG, "c_in=%d c_out=%d", d->c_in, d->c_out);
  if (d->ksize != 0 && d->ksize != 3)
    return api_fail(SNN_ERR_UNSUPPORTED, "the no-allocation entry point runs 3x3 layers only (ksize=%d)", d->ksize);
  if (d->tau < 1 || d->tau > 9) return api_fail(SNN_ERR_INVALID_ARG, "tau=%d outside 1..9", d->tau);
  if (d->stride < 1 || d->stride > 2) return api_fail(SNN_ERR_INVALID_ARG, "stride=%d outside {1,2}", d->stride);
  if (d->pad < 0 || d->pad > 1) return api_fail(SNN_ERR_INVALID_ARG, "pad=%d outside {0,1}", d->pad);
  if (d->act_type != SNN_ACT_BIN)
    return api_fail(SNN_ERR_UNSUPPORTED, "the no-allocation entry point takes binary activations only");
  if (out_type != SNN_OUT_F32 && out_type != SNN_OUT_I32) return api_fail(SNN_ERR_INVALID_ARG, "bad out_type %d", out_type);
  if (d->c_in > SNN_STATIC_MAX_CHANNELS || d->c_out > SNN_STATIC_MAX_CHANNELS)
    return api_fail(SNN_ERR_UNSUPPORTED, "c_in=%d / c_out=%d exceed the no-allocation limit of %d channels", d->c_in,
                    d->c_out, SNN_STATIC_MAX_CHANNELS);
  const int T = 1 << d->tau;
  for (int j = 0; j < T; ++j)
    if (d->codebook[j] >= 512) return api_fail(SNN_ERR_INVALID_ARG, "codebook[%d]=%u is not a 9-bit code", j, d->codebook[j]);
  for (int k = 0; k < d->c_out; ++k)
    if (!std::isfinite(d->alpha[k])) return api_fail(SNN_ERR_INVALID_ARG, "alpha[%d] is not finite", k);
  if (N < 0 || H < 1 || W < 1 || H + 2 * d->pad < 3 || W + 2 * d->pad < 3)
    return api_fail(SNN_ERR_INVALID_ARG, "shape N=%d H=%d W=%d gives no output", N, H, W);
  if (N == 0) return SNN_OK;
  if (!act_dev || !out_dev) return api_fail(SNN_ERR_INVALID_ARG, "null activation / output pointer");
  if (((uintptr_t)act_dev & 15) || ((uintptr_t)out_dev & 15))
    return api_fail(SNN_ERR_INVALID_ARG, "activation / output pointers must be 16-byte aligned");

  Geom g;
  g.N = N; g.H = H; g.W = W;
  g.C = d->c_in; g.K = d->c_out; g.Cw = (d->c_in + 31) / 32;
  g.stride = d->stride; g.pad = d->pad;
  g.Ho = (H + 2 * d->pad - 3) / d->stride + 1;
  g.Wo = (W + 2 * d->pad - 3) / d->stride + 1;
  g.tau = d->tau; g.T = T;
  if ((long long)N * H * W >= (1ll << 31) || (long long)N * g.Ho * g.Wo >= (1ll << 31))
    return api_fail(SNN_ERR_INVALID_ARG, "shape too large");

  // ---- carve the fixed array; refuse what does not fit
  const size_t n_elem = (size_t)g.K * g.C;
  const size_t stream_bytes = (n_elem * g.tau + 7) / 8;
  const int Tp = (T + 15) / 16 * 16;
  size_t off = 0;
  const size_t o_stream = off;  off = align256(off + stream_bytes + 4);
  const size_t o_idx = off;     off = align256(off + n_elem * 2);
  const size_t o_cb = off;      off = align256(off + (size_t)T * 2);
  const size_t o_alpha = off;   off = align256(off + (size_t)g.K * 4);
  const size_t o_planes = off;  off = align256(off + (size_t)9 * g.Cw * g.K * 4);
  const size_t o_corr = off;    off = align256(off + (size_t)16 * g.K * 4);
  const size_t o_match = off;   off = align256(off + (size_t)Tp * 512);
  if (off > kStaticScratchBytes)
    return api_fail(SNN_ERR_UNSUPPORTED, "layer needs %zu bytes of scratch, the fixed array holds %zu", off,
                    kStaticScratchBytes);

  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
    cudaGetLastError();
    return api_fail(SNN_ERR_CUDA, "no CUDA device available (this library has no CPU path)");
  }
  if (d->device < 0 || d->device >= ndev || d->device >= kMaxDevices)
    return api_fail(SNN_ERR_INVALID_ARG, "device %d of %d", d->device, ndev);
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != d->device && cudaSetDevice(d->device) != cudaSuccess)
    return api_fail(SNN_ERR_CUDA, "cannot select device %d", d->device);

  snn_status_t st = SNN_OK;
  unsigned char* base = nullptr;
  cudaError_t e = scratch_address(d->device, &base);  // first call on a device resolves the symbol
  cudaStream_t s = (cudaStream_t)cuda_stream;
  LayerDev L;
  if (e == cudaSuccess) {
    L.idx = reinterpret_cast<uint16_t*>(base + o_idx);
    L.codebook = reinterpret_cast<uint16_t*>(base + o_cb);
    L.alpha = reinterpret_cast<float*>(base + o_alpha);
    L.wplanes = reinterpret_cast<uint32_t*>(base + o_planes);
    L.corr = reinterpret_cast<int32_t*>(base + o_corr);
    L.match9 = base + o_match;
    e = cudaMemcpyAsync(base + o_stream, d->idx_packed, stream_bytes, cudaMemcpyHostToDevice, s);
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(L.codebook, d->codebook, (size_t)T * 2, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(L.alpha, d->alpha, (size_t)g.K * 4, cudaMemcpyHostToDevice, s);
  int launched = 0;
  // every region the kernels read is rewritten in full by this call, so nothing left
  // behind by the previous call can leak into the result and nothing needs clearing
  if (e == cudaSuccess) e = decode_layer(L, base + o_stream, g, SNN_ACT_BIN, s, &launched);
  if (e == cudaSuccess) {
    Launch l{act_dev, out_dev, out_type == SNN_OUT_I32, s};
    e = popc_forward(L, g, l, &launched);
  }
  api_count_launches(launched);
  if (e != cudaSuccess) st = api_fail(SNN_ERR_CUDA, "snn_conv_forward_static: %s", cudaGetErrorString(e));
  if (prev >= 0 && prev != d->device) cudaSetDevice(prev);
  return st;
}
