/*
 * eas_encoder.h -- C ABI of the Encode-stage library (sm_100a).
 *
 * The paper makes the Encode stage (modality encoder plus connector, Section 2.1) the control
 * point of an Encode-Prefill-Decode serving pipeline: requests are grouped into load-adaptive
 * micro-batches (Section 3.2), each micro-batch is ONE encoder forward pass, and the pass runs
 * on a share of the GPU's SMs chosen per micro-batch (Section 3.4).  This library is that forward
 * pass: a micro-batch of media items in, one embedding block per item out, on `sm_budget` SMs.
 * Encoder families follow Table 3 (CLIP-style ViT, dynamic-resolution ViT, Whisper-style audio).
 *
 * Conventions
 *  - Every pointer says "device" or "host".  All device buffers (weights, arena, inputs, workspace,
 *    outputs) are allocated and freed by the caller; the library allocates no device memory.
 *  - bf16 = IEEE bfloat16 bit patterns.  Linear weights are row-major [out_features, in_features].
 *  - Calls return an eas_status; nothing throws or aborts.  eas_last_error() gives a thread-local text.
 *  - eas_encode_microbatch only enqueues work on `stream`; outputs are valid once the stream has
 *    reached that point.  Host arrays may be reused as soon as the call returns.
 *  - Results are deterministic: the same inputs give the same bytes for any sm_budget and any packing.
 *  - One handle serves one call at a time; different handles are independent.
 */
#ifndef EAS_ENCODER_H_
#define EAS_ENCODER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct eas_encoder eas_encoder; /* opaque */

typedef enum {
  EAS_OK = 0,
  EAS_ERR_INVALID_ARG = 1,    /* null pointer, bad size, inconsistent shapes; nothing was launched */
  EAS_ERR_UNSUPPORTED = 2,    /* a valid request this build has no kernel for (e.g. head_dim not 64/80) */
  EAS_ERR_WORKSPACE = 3,      /* workspace or weight arena too small */
  EAS_ERR_CUDA = 4,           /* a CUDA runtime call failed (text in eas_last_error) */
  EAS_ERR_DEVICE_TIMEOUT = 5, /* a bounded device-side wait expired; outputs of that call are invalid */
  EAS_ERR_ARCH = 6,           /* the current device is not compute capability 10.x */
  EAS_ERR_DEVICE_CHECK = 7    /* a device-side consistency check failed (e.g. device cu_seqlens != host copy) */
} eas_status;

enum { EAS_FAMILY_VIT_LEARNED = 0, EAS_FAMILY_VIT_ROPE_MERGER = 1, EAS_FAMILY_AUDIO_CONV = 2 };
enum { EAS_NORM_LAYERNORM = 0, EAS_NORM_RMSNORM = 1 };
enum { EAS_MLP_GELU = 0, EAS_MLP_SWIGLU = 1 };
enum { EAS_POS_TABLE = 0, EAS_POS_ROPE_2D = 1 };
enum { EAS_HEAD_NONE = 0, EAS_HEAD_MLP_PROJECTOR = 1, EAS_HEAD_MERGER_2X2 = 2 };
enum { EAS_OUT_BF16 = 0, EAS_OUT_FP32 = 1 };
enum { EAS_MAX_ITEMS = 128 }; /* items per micro-batch */

/* Architecture record (plain data, copied at create).  Encoder = embedding front end, n_layers
 * pre-norm transformer blocks, connector ("head").  Table 3 names the families; the numbers are
 * the caller's. */
typedef struct {
  int32_t family;         /* EAS_FAMILY_* : patch embedding + position table | patch embedding + 2-D rotary
                             + 2x2 merger | two k=3 convolutions (stride 1, 2) + position table */
  int32_t n_layers, d_model, n_heads, d_mlp; /* d_model % n_heads == 0; head_dim in {64, 80}; d_model % 128 == 0 */
  int32_t norm;           /* EAS_NORM_* */
  float   norm_eps;
  int32_t mlp;            /* EAS_MLP_GELU: fc2(GELU_erf(fc1 x)); EAS_MLP_SWIGLU: fc2(SiLU(gate x) * up x) */
  int32_t in_channels;    /* image channels; audio: mel bins */
  int32_t patch;          /* spatial patch edge (audio: 1) */
  int32_t temporal_patch; /* frames per patch (1 for images) */
  int32_t has_cls;        /* prepend a learned CLS token per item */
  int32_t embed_norm;     /* normalise the residual stream right after the embedding */
  int32_t final_norm;     /* normalise after the last block */
  int32_t pos;            /* EAS_POS_* */
  int32_t max_pos;        /* rows of the position table */
  float   rope_theta;
  int32_t head;           /* EAS_HEAD_* */
  int32_t d_head_hidden;  /* hidden width of the connector MLP */
  int32_t d_out;          /* embedding width delivered to the LLM */
  int32_t out_dtype;      /* EAS_OUT_BF16 (default): out_embeddings is bf16.  EAS_OUT_FP32: the last kernel (final norm or
                             the connector's second GEMM) writes its fp32 result unrounded, out_embeddings is fp32
                             [out_rows, d_out]: for consumers that want the embeddings without the 2^-9 output rounding */
} eas_arch_config;

/* One named weight tensor in device memory, bf16.
 * Names: embed.w [d, C*pt*P*P] (patch element order: channel, frame-in-patch, row, column), embed.b;
 * audio: conv1.w [d,3,n_mel], conv1.b, conv2.w [d,3,d], conv2.b (tap-major, then channel);
 * cls [d]; pos [max_pos,d]; embed_norm.{g,b}; blk{i}.norm1.{g,b}; blk{i}.qkv.{w [3d,d], b} (rows: all Q, all K,
 * all V; head h owns rows h*head_dim.. of each third); blk{i}.proj.{w,b}; blk{i}.norm2.{g,b}; blk{i}.fc1.{w [I,d], b}
 * or blk{i}.gate.{w,b} + blk{i}.up.{w,b}; blk{i}.fc2.{w [d,I], b}; final_norm.{g,b}; head.norm.g; head.fc1.{w,b};
 * head.fc2.{w,b}.  RMSNorm has no ".b". */
typedef struct {
  const char* name;    /* host */
  const void* dev_ptr; /* device, bf16, 16-byte aligned, contiguous */
  int32_t ndim;
  int64_t shape[4];
} eas_tensor;

typedef struct {
  const eas_tensor* tensors; /* host array */
  int32_t n_tensors;
  void* arena;               /* device scratch of eas_encoder_weight_arena_bytes(): the library re-lays some
                                weights into it at create (padded patch matrix, rotary row pairing, gate/up
                                interleave).  Caller-owned; must outlive the handle, as must the weights. */
  size_t arena_bytes;
} eas_weights;

/* One micro-batch (Section 3.2: the unit of one forward pass). */
typedef struct {
  const void* data;               /* device, bf16, items back to back.  Image [C,H,W]; clip [F,C,H,W]; audio [frames, mel] */
  int32_t n_items;                /* 1..EAS_MAX_ITEMS */
  const int32_t* item_shape;      /* host [n_items][3]: (frames, height, width); audio: (n_frames, n_mel, 1), any
                                     n_frames >= 1: the stride-2 convolution yields ceil(n_frames / 2) tokens */
  const int64_t* item_offset;     /* host [n_items]: element offset of each item in data */
  const int32_t* cu_seqlens_host; /* host [n_items+1]: prefix sums of ENCODER tokens per item (after patching or
                                     convolution, CLS included); checked against item_shape */
  void* workspace;                /* device scratch of eas_encoder_workspace_bytes(); 1024-byte aligned */
  size_t workspace_bytes;
} eas_packed_inputs;

/* Section 2.1 (encoder + connector).  Validates the record, locates the weights, re-lays what the kernels
 * need into weights->arena (launches small kernels on the legacy default stream and synchronises).
 * Errors: INVALID_ARG (missing/misshaped tensor, bad record), UNSUPPORTED, WORKSPACE (arena too small),
 * ARCH, CUDA.  *out is NULL on error. */
eas_status eas_encoder_create(const eas_arch_config* arch, const eas_weights* weights, eas_encoder** out);

/* Bytes of device arena eas_encoder_create needs for this architecture (0 on a bad record). */
size_t eas_encoder_weight_arena_bytes(const eas_arch_config* arch);

/* Bytes of device workspace for a micro-batch of n_items items with total_tokens encoder tokens. */
size_t eas_encoder_workspace_bytes(const eas_encoder* enc, int64_t total_tokens, int32_t n_items, int32_t max_seqlen);

/* Output rows the micro-batch will produce (sum over items: tokens, tokens-1 with CLS + projector, tokens/4
 * with the merger); -1 on error. */
int64_t eas_encoder_out_rows(const eas_encoder* enc, const int32_t* cu_seqlens_host, int32_t n_items);

/* Sections 3.2 and 3.4: one encoder forward pass over a micro-batch on `sm_budget` SMs.
 * cu_seqlens: device int32 [n_items+1], same values as cu_seqlens_host (compared on the device; a mismatch
 *   raises EAS_ERR_DEVICE_CHECK at the next eas_encoder_status).  Items never attend across each other.
 * sm_budget: number of SMs every kernel of this call may occupy, 1..SM count; 0 = all.
 * stream: a cudaStream_t (NULL = legacy default stream).
 * out_embeddings: device bf16 (fp32 with EAS_OUT_FP32) [out_rows, d_out]; rows of item i start at the sum of earlier
 *   items' rows.
 * Errors (nothing launched): INVALID_ARG (null pointers, n_items out of range, non-monotone cu_seqlens,
 *   sizes not multiples of the patch / merge / temporal patch, tokens inconsistent with shapes, more tokens
 *   than position rows, sm_budget out of range), WORKSPACE. */
eas_status eas_encode_microbatch(eas_encoder* enc, const eas_packed_inputs* in, const int32_t* cu_seqlens,
                                 int32_t sm_budget, void* stream, void* out_embeddings);

/* The paper has no counterpart for this entry point; it exists for callers that cannot allocate device memory.
 * An encode worker that shares its GPU with a prefill worker (Section 3.4 co-locates them) typically starts after
 * the neighbour has claimed the rest of HBM for its KV cache, and runs inside a serving loop where an allocation may
 * fail, or may make the whole device wait while the driver grows its heap.  Such a caller can use this variant of
 * eas_encode_microbatch: same arguments, same result, but the scratch the forward pass needs comes from an array of
 * EAS_STATIC_WORKSPACE_BYTES that is part of the library image, so the call itself allocates nothing (no cudaMalloc,
 * cudaFree, or allocating library routine).  in->workspace and in->workspace_bytes are ignored; the caller still
 * provides data, cu_seqlens and out_embeddings.
 *  - Limit: the micro-batch must fit the built-in scratch.  The forward pass needs about
 *    14 * d_model + 2 * d_mlp + 2 * (patch elements, padded to 64) bytes per encoder token (fp32 residual stream, bf16
 *    normalised rows, Q|K|V, attention output, MLP activation, patch operand), i.e. about 7 KB per token for d_model = 256
 *    with d_mlp = 1024 and about 30 KB per token for d_model = 1280 with d_mlp = 5120; eas_encoder_workspace_bytes()
 *    gives the exact figure.  32 MiB hold about 4600 tokens of the former and 1100 of the latter.  A larger micro-batch
 *    is rejected with EAS_ERR_WORKSPACE and a message that states both sizes.
 *  - Cost: every GPU on which this library is loaded holds the array until the process exits.
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that device
 *    current).  Make that first call before starting any stream capture.
 *  - All calls on one device share the one array, which keeps whatever the previous call left in it.  The forward
 *    pass clears its status word itself and writes every other scratch region before reading it, so nothing has to
 *    be zeroed by the caller; but two calls whose kernels overlap on the GPU (different streams, or different
 *    handles) would race on it.  Serialise them, or use eas_encode_microbatch with separate workspaces. */
#define EAS_STATIC_WORKSPACE_BYTES (32u << 20)
eas_status eas_encode_microbatch_static(eas_encoder* enc, const eas_packed_inputs* in, const int32_t* cu_seqlens,
                                        int32_t sm_budget, void* stream, void* out_embeddings);

/* Synchronises `stream`, then reads and clears the device status word of the last call's workspace:
 * EAS_OK, EAS_ERR_DEVICE_TIMEOUT, EAS_ERR_DEVICE_CHECK or EAS_ERR_CUDA. */
eas_status eas_encoder_status(eas_encoder* enc, void* stream);

/* Number of kernel launches the last eas_encode_microbatch enqueued. */
int32_t eas_encoder_last_launch_count(const eas_encoder* enc);

/* Selects the attention kernel: 0 = default (tcgen05, probabilities kept in tensor memory); 1 = register-tile
 * (mma.sync) kernel; 2 = tcgen05 with the probabilities staged in shared memory.  1 and 2 are cross-checks for
 * testing. */
eas_status eas_encoder_set_attention_impl(eas_encoder* enc, int32_t impl);

/* Split K for small micro-batches (default off; part of the latency path, like the graph mode below).  With few tokens
 * the residual GEMMs of a block (x += o W_proj^T, x += h W_fc2^T) have fewer tiles than the device has SMs, and the K
 * loop of one tile is the whole kernel.  With on = 1, when tiles x s <= SMs and K / s >= 1024 (s = 4 or 2; a function of
 * the token count, the layer sizes and the device, never of sm_budget), s CTAs share a tile's K range: the first adds its
 * sum and the bias into the residual stream as usual, the others store bare partial sums, and the normalisation kernel
 * that follows adds those to the row in a fixed order before normalising it.  Results stay deterministic and independent
 * of sm_budget, but no longer of what else is in the micro-batch: an item encoded alone (split) and the same item in a
 * large micro-batch (not split) differ in the last bits, which is why the mode is off unless asked for (off: every
 * item's embeddings are bit-identical whatever it is packed with).  eas_encoder_workspace_bytes follows the mode (the
 * partial sums need scratch): set it before sizing the workspace. */
eas_status eas_encoder_set_split_k(eas_encoder* enc, int32_t on);

/* Folded normalisation (default on).  A block's norm1 / norm2 (Section 2.1: pre-norm transformer blocks) are followed by
 * a linear layer, and  LN(x) W^T + b  =  rstd * ((gamma .* x) W^T - mean (gamma W^T)) + (b + beta W^T):  the qkv and
 * MLP-up GEMMs run on the residual rows scaled by gamma only (rounded to bf16) and apply each row's rstd and mean in
 * their epilogue, with two constants per output computed at create time, so no normalisation kernel runs inside a block.  The rows' statistics (mean
 * and squared deviations per 128 columns, merged in index order: independent of sm_budget and of the tile shape) and
 * their scaled bf16 copy are written by the residual GEMM that produced the rows, in the same pass that adds into the fp32
 * stream.  on = 0 restores one normalisation kernel per norm1 / norm2 (the result differs in rounding only: the
 * normalised values are then rounded to bf16 before the GEMM instead of the scaled ones).  While split K is in effect for a
 * micro-batch its blocks run unfolded.  Both modes stay within the same parity tolerance of the definition. */
eas_status eas_encoder_set_norm_fold(eas_encoder* enc, int32_t on);

/* Launch-overhead path for small micro-batches (Section 3.2: a forward pass at small batch size is dominated by
 * kernel-launch and scheduling overhead).  mode 1: eas_encode_microbatch / _static capture the launches of a
 * micro-batch into a CUDA graph the first time they see it and replay the graph afterwards (one driver call per
 * forward pass instead of one per kernel).  A micro-batch is "the same" when n_items, item_shape, item_offset,
 * cu_seqlens_host, sm_budget, the attention variant and every pointer (data, workspace, cu_seqlens_dev,
 * out_embeddings) are equal; the VALUES behind the pointers may change freely.  The kernels and their arguments are
 * those of the ordinary path, so results are bit-identical.  Up to 16 captures are kept per encoder (least recently
 * used goes first); mode 0 (default) drops them.  Capture needs a real stream: with the NULL / legacy / per-thread
 * default stream, while per-kernel timing is on, or while the caller is itself capturing `stream`, calls run
 * uncaptured.  The cached graphs refer to the caller's buffers: do not free those while the mode is on. */
eas_status eas_encoder_set_graph_mode(eas_encoder* enc, int32_t mode);

/* Counters of the graph path: replays, captures, and captures currently held (any pointer may be NULL). */
eas_status eas_encoder_graph_stats(const eas_encoder* enc, int64_t* hits, int64_t* captures, int32_t* cached);

/* Per-kernel timing for profiling (off by default; adds one event record per launch).  Kernel classes: */
enum { EAS_KC_PREP = 0, EAS_KC_EMBED_GATHER = 1, EAS_KC_GEMM_EMBED = 2, EAS_KC_NORM = 3, EAS_KC_GEMM_QKV = 4,
       EAS_KC_ATTENTION = 5, EAS_KC_GEMM_PROJ = 6, EAS_KC_GEMM_FC1 = 7, EAS_KC_GEMM_FC2 = 8, EAS_KC_GEMM_HEAD = 9,
       EAS_KC_COUNT = 10 };
/* on != 0: the following eas_encode_microbatch calls record a CUDA event in front of every launch. */
eas_status eas_encoder_enable_timing(eas_encoder* enc, int32_t on);
/* Waits for the last timed call, then writes the class and device milliseconds of its launches, in launch
 * order, into host arrays of `capacity` entries.  Returns the number written (with NULL arrays: the number
 * available), or -1 on a CUDA error. */
int32_t eas_encoder_timing_read(eas_encoder* enc, int32_t capacity, int32_t* kernel_class, float* ms);

/* ---- SM partition (Section 3.4: the encoder gets a share of the SMs, the co-located prefill worker the rest) ----
 * eas_sm_partition_create splits the current device's SMs into two disjoint sets with the driver's green contexts
 * and creates one non-blocking stream in each: side 0 holds at least `sm_encode` SMs (the driver rounds up to its
 * granularity, 8 SMs on this architecture, and keeps SM pairs together so that CTA-pair clusters still launch), side 1
 * the remaining ones.  Kernels enqueued on a side's stream run only on that side's SMs, whatever their grid size, so an
 * encoder call given side 0's stream and sm_budget = eas_sm_partition_sm_count(p, 0) cannot be slowed by a neighbour's
 * kernels occupying its SMs; L2 and HBM stay shared.  Device memory is shared with the rest of the process.
 * Errors: EAS_ERR_INVALID_ARG (sm_encode <= 0 or nothing left for side 1), EAS_ERR_UNSUPPORTED (driver without
 * green contexts), EAS_ERR_CUDA.  The handle owns the streams and contexts: destroy it after the work on them is done
 * (destroy waits for both streams). */
typedef struct eas_sm_partition eas_sm_partition;
eas_status eas_sm_partition_create(int32_t sm_encode, eas_sm_partition** out);
/* Number of SMs of side 0 (encoder) or 1 (neighbour); 0 for any other argument. */
int32_t eas_sm_partition_sm_count(const eas_sm_partition* p, int32_t side);
/* The side's stream (a cudaStream_t), owned by the handle. */
void* eas_sm_partition_stream(const eas_sm_partition* p, int32_t side);
void eas_sm_partition_destroy(eas_sm_partition* p);

const char* eas_last_error(void);

void eas_encoder_destroy(eas_encoder* enc);

/* ---- single-kernel entry points (the same kernels the encoder launches; used by tests and micro-benchmarks) ---- */

/* out[M, N or N/2] = epilogue(A[M,K] * W[N,K]^T + bias).  A, W, bias: device bf16; K % 64 == 0, N % 32 == 0.
 * act: 0 none, 1 GELU (erf), 2 SwiGLU (W rows and bias interleaved gate_0, up_0, gate_1, ...; out is [M, N/2]).
 * out_fp32: 0 -> bf16 out; 1 -> fp32 out, and resid (device fp32 [M,N], may equal out, may be NULL) is added.
 * status_dev: device uint32 the kernel raises on a bounded-wait expiry (caller zeroes it). */
eas_status eas_kernel_gemm(const void* A, const void* W, const void* bias, void* out, const float* resid,
                           int32_t M, int32_t N, int32_t K, int32_t act, int32_t out_fp32, int32_t sm_budget,
                           void* stream, uint32_t* status_dev);

/* The same call with the tile shape fixed instead of chosen by the launcher's cost model: 0 = choose (as above),
 * 1 = one CTA per 128x256 tile, 2 = a CTA pair per 256x256 tile, 3 = a CTA pair per 256x512 tile (needs N % 512 == 0,
 * act 0 or 1; EAS_ERR_UNSUPPORTED otherwise).  All shapes accumulate over K in the same order, so their results are
 * bit-identical; the tests use this to check exactly that.  With sm_budget 1 only shape 1 exists and the argument is
 * ignored. */
eas_status eas_kernel_gemm_tile(const void* A, const void* W, const void* bias, void* out, const float* resid,
                                int32_t M, int32_t N, int32_t K, int32_t act, int32_t out_fp32, int32_t sm_budget,
                                void* stream, uint32_t* status_dev, int32_t tile_shape);

/* y[rows,d] = norm(x[rows,d]): kind 0 LayerNorm (gamma, beta), 1 RMSNorm (gamma), 2 plain cast.  x device fp32;
 * gamma/beta device bf16; y device bf16 (out_fp32 = 0) or fp32.  d % 128 == 0, d <= 2048. */
eas_status eas_kernel_norm(const float* x, void* y, const void* gamma, const void* beta, int32_t rows, int32_t d,
                           int32_t kind, float eps, int32_t out_fp32, int32_t sm_budget, void* stream);

/* Block-diagonal attention over packed qkv (device bf16 [T, 3*n_heads*head_dim], thirds Q|K|V) -> out (device
 * bf16 [T, n_heads*head_dim]).  cu_seqlens_host: host int32 [n_items+1].  impl as in eas_encoder_set_attention_impl. */
eas_status eas_kernel_attention(const void* qkv, void* out, const int32_t* cu_seqlens_host, int32_t n_items,
                                int32_t n_heads, int32_t head_dim, int32_t sm_budget, void* stream, int32_t impl,
                                uint32_t* status_dev);

#ifdef __cplusplus
}
#endif
#endif /* EAS_ENCODER_H_ */
