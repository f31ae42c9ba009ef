/*
 * snn_conv.h -- C ABI of the sub-bit binary 3x3 convolution library (sm_100a).
 *
 * One layer of a Sub-bit Neural Network is stored as (Sec. 4.4 "Compression"):
 * a layer-specific set of 2^tau binary 3x3 kernels (the codebook), one tau-bit
 * index per (c_out, c_in) kernel, and channel-wise scales (Sec. 3).  Its
 * forward pass is  Y = alpha * (w_bar o a_bar)  (Sec. 3; Algorithm 1, forward
 * step), a 3x3 cross-correlation of +/-1 weights with +/-1 activations, or
 * with fp16 activations in the weights-only setting (Sec. 5.3 deployment test,
 * Table 2 ".../32" rows).
 *
 * Conventions fixed by this library:
 *   - code of a kernel: 9-bit integer, bit (8 - (3*ky + kx)) set <=> K[ky][kx] = +1.
 *     Code 0 is the all -1 kernel (the paper's kernel no. 1), code 511 the
 *     all +1 kernel (no. 512) (Sec. 4.1).  Everything is 0-based here.
 *   - index stream: element e = co*c_in + ci occupies bits [e*tau, (e+1)*tau) of
 *     an LSB-first byte stream (tau*c_in*c_out bits in total, Sec. 4.4).
 *   - binary activations: uint32 [N][H][W][ceil(c_in/32)], channel ci = bit ci%32
 *     of word ci/32, bit 1 = +1, bit 0 = -1, unused high bits MUST be 0.
 *   - fp16 activations: IEEE binary16 [N][H][W][c_in].
 *   - output: [N][Ho][Wo][c_out], Ho = floor((H + 2*pad - 3)/stride) + 1,
 *     int32 pre-scale sums S or fp32 Y = (float)S * alpha[co] (one multiply).
 *   - zero padding contributes 0 to the sum (it is not a -1).
 *
 * All entry points return a status; on failure snn_last_error() gives a text.
 * Nothing throws, aborts or traps.  There is no CPU fallback: every step runs
 * in CUDA kernels, and a path that does not support a shape says so.
 */
#ifndef SNN_CONV_H_
#define SNN_CONV_H_

#include <stdint.h>

#if defined(__GNUC__)
#define SNN_API __attribute__((visibility("default")))
#else
#define SNN_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct snn_conv snn_conv_t; /* opaque; owned by the library */

typedef enum {
  SNN_OK = 0,
  SNN_ERR_INVALID_ARG = 1,
  SNN_ERR_UNSUPPORTED = 2, /* path cannot run this shape; nothing was launched */
  SNN_ERR_CUDA = 3,
  SNN_ERR_OOM = 4,
  SNN_ERR_TIMEOUT = 5      /* a bounded device-side wait ran out */
} snn_status_t;

enum { SNN_ACT_BIN = 0, SNN_ACT_F16 = 1 };
enum {
  SNN_OUT_F32 = 0,
  SNN_OUT_I32 = 1,  /* only with SNN_ACT_BIN */
  SNN_OUT_BITS = 2  /* only with SNN_ACT_BIN and the tensor-core path: the thresholded signs of Y, packed as the
                       next layer's binary input (Algorithm 1: layer i consumes sign(a^{i-1}); between two
                       binary layers sit a batch normalisation and a Hardtanh, Sec. 5, i.e. a per-channel
                       affine map whose sign is the sign of Y plus a per-channel constant):
                       uint32 [N][Ho][Wo][ceil(c_out/32)], bit co%32 of word co/32 = 1 iff
                       fl(fl(alpha[co] * S) + shift[co]) >= 0 in fp32, round to nearest even
                       (so 0 gives +1; shift is 0 where the descriptor has none), unused high bits 0 */
};
enum {
  SNN_PATH_AUTO = 0,       /* tuned choice if snn_conv_tune ran for the shape, else a heuristic */
  SNN_PATH_REUSE = 1,      /* codebook-reuse: per-channel partial maps + index-driven accumulate (Sec. 4.5);
                              binary activations, or fp16 activations with at most 1024 output channels */
  SNN_PATH_DECODED = 2,    /* decoded weights, XOR + popcount implicit GEMM (Sec. 3); binary activations */
  SNN_PATH_DECODED_TC = 3  /* decoded weights on the tcgen05 tensor cores */
};

typedef struct {
  int32_t c_in, c_out;        /* >= 1; need not be multiples of 32 */
  int32_t tau;                /* 1..9; 9 = full 512-kernel codebook = a standard 1-bit layer (Sec. 4.1) */
  int32_t stride, pad;        /* stride in {1,2}; pad in {0,1}; kernel is 3x3 */
  int32_t act_type;           /* SNN_ACT_* */
  int32_t device;             /* CUDA ordinal */
  const uint16_t* codebook;   /* HOST, 2^tau codes, each < 512; duplicates allowed */
  const uint8_t* idx_packed;  /* HOST, ceil(c_out*c_in*tau/8) bytes, see above */
  const float* alpha;         /* HOST, c_out finite fp32 scales */
  const float* shift;         /* HOST, c_out finite fp32 thresholds added to Y before its sign is taken
                                 (SNN_OUT_BITS only; fp32 and int32 outputs ignore it), or NULL for none */
  int32_t ksize;              /* 0 or 3: a 3x3 layer as above.  1: the 1x1 extension (appendix "Extending to
                                 Bottleneck with 1x1 Kernels"): the weights are c_out * c_in/8 vectors of 8
                                 consecutive input channels, each a tau-bit index (1 <= tau <= 8) into a set of
                                 2^tau 8-bit codes (each < 256; bit 7 - j set <=> element j, i.e. channel 8g + j,
                                 is +1; code 0 all -1, code 255 all +1); index element e = co*(c_in/8) + g;
                                 c_in divisible by 8, pad 0, Ho = floor((H - 1)/stride) + 1.  Only the
                                 tensor-core path runs such a layer. */
} snn_conv_desc_t;

/*
 * Sec. 4.4 storage -> device form.  Copies the host arrays (the caller may free
 * them on return), unpacks the index stream and decodes the weights on the
 * device.  *out receives a handle that owns its device buffers.
 * Errors: INVALID_ARG (null pointer, tau/stride/pad out of range, code >= 512,
 * non-finite alpha or shift, c_in/c_out < 1), CUDA, OOM.
 */
SNN_API snn_status_t snn_conv_create(const snn_conv_desc_t* desc, snn_conv_t** out);

/*
 * Sec. 3 / Algorithm 1 forward step for one batch.  act_dev and out_dev are
 * DEVICE pointers owned by the caller (layouts above), act_dev 16-byte aligned,
 * out_dev 16-byte aligned; they are neither kept nor freed.  The call is
 * asynchronous on cuda_stream (a cudaStream_t, NULL = default stream) and does
 * not allocate, with one exception: the tensor-core path builds its plan and its
 * tiled weight operand (device memory owned by the handle) at the first call for
 * an input shape and output kind, so make that first call outside stream capture
 * (snn_conv_tune for the shape does it for fp32 and int32 outputs).  N may be 0
 * (nothing is launched).
 * Errors: INVALID_ARG (null, H/W giving no output, I32 or BITS output with fp16
 * activations, unknown path), UNSUPPORTED (the named path cannot run this
 * layer; AUTO never returns it, except for SNN_OUT_BITS on a layer the
 * tensor-core path cannot run), CUDA.
 */
SNN_API snn_status_t snn_conv_forward(snn_conv_t* h, const void* act_dev, int32_t N, int32_t H, int32_t W,
                              void* out_dev, int32_t out_type, int32_t path, void* cuda_stream);

/*
 * Same operation with HOST buffers: copies act_host to the device, runs the
 * forward pass, copies the result back and waits for it.  Staging buffers live
 * in the handle and grow on demand (the only call besides create/tune that may
 * allocate).  Pinned host memory makes the copies asynchronous.
 */
SNN_API snn_status_t snn_conv_forward_host(snn_conv_t* h, const void* act_host, int32_t N, int32_t H, int32_t W,
                                   void* out_host, int32_t out_type, int32_t path);

/*
 * Path selection from measured time (Sec. 4.5: the gain of sharing depends on
 * 2^tau / c_out, so the choice is per layer shape).  Times every supported
 * path on zero-filled scratch inputs of the given shape and remembers the
 * fastest for (N, H, W).  Synchronous.  *best_path / ms[4] (indexed by
 * SNN_PATH_*, negative = unsupported) may be NULL.
 */
SNN_API snn_status_t snn_conv_tune(snn_conv_t* h, int32_t N, int32_t H, int32_t W, int32_t* best_path, float* ms);

/* Path SNN_PATH_AUTO would take for this shape (never AUTO itself). */
SNN_API int32_t snn_conv_chosen_path(const snn_conv_t* h, int32_t N, int32_t H, int32_t W);

/* SNN_OK if `path` can run this layer at this shape, else SNN_ERR_UNSUPPORTED. */
SNN_API snn_status_t snn_conv_path_supported(const snn_conv_t* h, int32_t path, int32_t N, int32_t H, int32_t W);

/* Frees the handle and its device buffers.  NULL is a no-op returning SNN_OK. */
SNN_API snn_status_t snn_conv_destroy(snn_conv_t* h);

/* Text of the calling thread's last failure; never NULL. */
SNN_API const char* snn_last_error(void);

SNN_API const char* snn_version(void);

/* Number of kernels this library has launched in this process (all handles). */
SNN_API int64_t snn_kernel_launches(void);

/*
 * Measured instruction-rate ceilings used as roofline denominators for the
 * ALU paths: runs a short saturating loop of one instruction kind on `device`
 * and returns results per second in *rate (per-lane results: a warp
 * instruction counts 32).  kind: 0 = POPC, 1 = LOP3 (xor), 2 = IADD3,
 * 3 = LDS.32 (conflict-free), 4 = XOR+POPC+IADD chain as the decoded loop issues it.
 * Ceilings of the tensor-core path, measured the way that path uses the hardware:
 * 5 = tcgen05.mma with 4-bit e2m1 operands and unit block scales (M = 128, N = 240,
 * K = 64, both operands from shared memory), in multiply-accumulates per second over
 * all SMs; 8 = the same at N = 128; 7 = tcgen05.mma with fp16 operands (M = 128,
 * N = 256, K = 16); 6 = a write-only stream of 16-byte stores over 1 GiB, in bytes
 * per second (the path writes 29 bytes for every byte it reads).
 * 9 = self-test of the bounded device-side waits, not a rate: one thread waits, with the
 * helper every kernel of the library waits with, on a barrier nothing ever arrives on.  The
 * wait must give up at its attempt limit and raise the status word the host reads, after
 * which the kernel ends normally: the call returns SNN_ERR_TIMEOUT (the expected outcome)
 * with *rate = the seconds the kernel took (about a second), and the device stays usable.
 * Any other return value means the mechanism is broken.
 */
SNN_API snn_status_t snn_microbench(int32_t kind, int32_t device, double* rate);

/*
 * A group of independent layer problems run as ONE persistent tensor-core launch.
 * The paper times whole networks (Sec. 5.3, Table 4: all binary layers of
 * ResNet-18/34 in one run); each member of a group is still the forward step of
 * Sec. 3 / Algorithm 1 for one layer, on that layer's own input, and the members
 * must not depend on each other (no member's output is another member's input
 * within one call): the CTAs walk through all members without any grid-wide step
 * in between, so that one member's start-up, first loads and last drain run beside
 * its neighbours' MMAs.
 *
 * snn_conv_group_create: `layers` are `count` (1..SNN_GROUP_MAX) handles of one
 * activation type on one device; N[i], H[i], W[i] fix the input shape of member i.
 * The group keeps the handles' device data by reference: the handles must outlive
 * the group.  It builds its own tiled weight operands (device memory owned by the
 * group), one set per output kind (words, packed signs): the tile shapes the kernel
 * is planned with differ between the two.  Errors: INVALID_ARG (null, count out of range, mixed activation types
 * or devices, a shape giving no output), UNSUPPORTED (a member the tensor-core
 * path cannot run; nothing is kept), CUDA, OOM.
 *
 * snn_conv_group_forward: act_dev[i] / out_dev[i] are HOST arrays of `count`
 * DEVICE pointers with the layouts and alignment of snn_conv_forward; outputs of
 * different members must not overlap.  out_type SNN_OUT_BITS writes the packed
 * signs instead (1 bit per output instead of 32; out_dev[i] 16-byte aligned as
 * well).  Asynchronous on cuda_stream; allocates nothing.  Errors: INVALID_ARG,
 * TIMEOUT (an earlier launch of the group gave up a bounded wait), CUDA.
 */
#define SNN_GROUP_MAX 32
typedef struct snn_conv_group snn_conv_group_t; /* opaque; owned by the library */
SNN_API snn_status_t snn_conv_group_create(snn_conv_t* const* layers, int32_t count, const int32_t* N,
                                           const int32_t* H, const int32_t* W, snn_conv_group_t** out);
SNN_API snn_status_t snn_conv_group_forward(snn_conv_group_t* g, const void* const* act_dev, void* const* out_dev,
                                            int32_t out_type, void* cuda_stream);
/* Frees the group and its device buffers (not the member handles).  NULL is a no-op. */
SNN_API snn_status_t snn_conv_group_destroy(snn_conv_group_t* g);

/*
 * A stack of layers that feed one another, run as ONE persistent tensor-core launch.
 * The paper times whole networks (Sec. 5.3, Table 4); in a binary network layer i + 1
 * consumes sign(a^i) (Algorithm 1, forward step), so the members of a stack are chained
 * through their packed thresholded signs (SNN_OUT_BITS: bit = fl(fl(alpha*S) + shift) >= 0,
 * shift standing for the batch normalisation / Hardtanh between two binary layers, Sec. 5):
 * member i writes them into a buffer the stack owns and member i + 1 reads them as its
 * binary input.  Shortcut additions are not part of the path.  Inside the launch a tile of
 * member i + 1 starts as soon as the tiles of member i that hold its input pixels are
 * complete (per-tile completion counters in device memory, every wait bounded); there is
 * no grid-wide step between layers.
 *
 * snn_conv_stack_create: `layers` are `count` (1..SNN_GROUP_MAX) handles with binary
 * activations on one device whose shapes follow from one another (c_in of member i + 1 =
 * c_out of member i, its input map = member i's output map); N, H, W fix the input of
 * member 0.  The handles must outlive the stack.  The stack owns the buffers between its
 * members, the counters and its tiled weight operands.  Errors: INVALID_ARG (null, count,
 * fp16 activations, shapes that do not chain, mixed devices), UNSUPPORTED (a member the
 * tensor-core path cannot run), CUDA, OOM.
 *
 * snn_conv_stack_forward: act_dev is member 0's input (DEVICE, binary layout), out_dev the
 * last member's output (DEVICE) of type out_type (SNN_OUT_F32, SNN_OUT_I32 or SNN_OUT_BITS);
 * both 16-byte aligned, neither kept.  Asynchronous on cuda_stream; allocates nothing.  Calls
 * on one stack must not overlap on the GPU (they share the buffers and counters).  All CTAs
 * of the launch must be resident together, which the launch checks (CUDA error otherwise).
 * Errors: INVALID_ARG, TIMEOUT (an earlier launch gave up a bounded wait), CUDA.
 */
typedef struct snn_conv_stack snn_conv_stack_t; /* opaque; owned by the library */
SNN_API snn_status_t snn_conv_stack_create(snn_conv_t* const* layers, int32_t count, int32_t N, int32_t H, int32_t W,
                                           snn_conv_stack_t** out);
SNN_API snn_status_t snn_conv_stack_forward(snn_conv_stack_t* s, const void* act_dev, void* out_dev, int32_t out_type,
                                            void* cuda_stream);
/* Frees the stack and its device buffers (not the member handles).  NULL is a no-op. */
SNN_API snn_status_t snn_conv_stack_destroy(snn_conv_stack_t* s);

/*
 * Forward pass for callers that must not allocate device memory.  (The paper has
 * no counterpart to this entry point; it exists for how the library is embedded.)
 *
 * Some hosts cannot let a library call cudaMalloc: an application that has handed
 * the whole device to its own memory pool, a process whose memory budget is fixed
 * at start-up, or a latency-bound loop that cannot afford the device-wide
 * synchronisation an allocation may bring.  snn_conv_create allocates, so such
 * callers use this call instead: it takes the layer as the descriptor states it
 * (HOST arrays, as for snn_conv_create) together with the DEVICE activation and
 * output buffers, and does everything else - copy of the layer, decode, XOR +
 * popcount convolution - inside one fixed device array that is part of the
 * library image (SNN_STATIC_SCRATCH_BYTES on every GPU that loads the library,
 * held until the process exits).  It calls no cudaMalloc / cudaFree and no
 * allocating library routine.
 *
 * Limits: binary activations only; c_in and c_out at most SNN_STATIC_MAX_CHANNELS
 * (a 512 x 512 layer with any tau fits); a layer whose scratch need exceeds the
 * array is refused with SNN_ERR_UNSUPPORTED and a message that names both sizes.
 * Layouts, output types and argument errors are those of snn_conv_forward; the
 * work is asynchronous on cuda_stream once the host arrays have been handed to
 * the copy engine (keep them alive and unchanged until the stream has passed them
 * unless they are pageable memory, which the runtime stages before returning).
 *
 * The first call on a device resolves the device address of the array
 * (cudaGetSymbolAddress); make that first call outside any stream capture.
 * All calls on a device share the one array and it keeps the previous call's
 * contents: each call rewrites in full every region it reads, so results never
 * depend on an earlier call, but two calls whose GPU work overlaps (different
 * streams, or threads) race on it.  Serialise them.
 */
#define SNN_STATIC_SCRATCH_BYTES (1536 * 1024)
#define SNN_STATIC_MAX_CHANNELS 512
SNN_API snn_status_t snn_conv_forward_static(const snn_conv_desc_t* desc, const void* act_dev, int32_t N, int32_t H,
                                             int32_t W, void* out_dev, int32_t out_type, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SNN_CONV_H_ */
