/*
 * epara.h -- C ABI of the B200 categorized serving step.
 *
 * One "step" executes, on one GPU, the forward passes of every admitted request of every
 * co-resident model: the single-GPU combination of the paper's allocation operators
 * batching (BS), multi-task (MT) and multi-frame (MF) (paper Section 3.1, "Allocation
 * operators") for the two categories that need no multi-GPU collaboration (Section 3.1,
 * "Performing operators to categories", first and third case).
 *
 * Ownership: the caller owns every byte of device memory (weights, KV pool, inputs,
 * outputs, workspace) and the CUDA stream.  The library borrows the pointers; they must
 * stay valid until the request is collected (weights/KV/workspace: until epara_destroy).
 * The library owns only host structures and its pinned descriptor buffers.
 *
 * Pointers named "device" are CUDA device pointers, 16-byte aligned; "host" pointers are
 * ordinary host memory read during the call only.  All tensors are row-major.  bf16 means
 * the upper 16 bits of an IEEE fp32.
 *
 * Errors: every function returns an epara_status; nothing throws, aborts or prints.
 * A context is not thread-safe: one host thread per context.
 */
#ifndef EPARA_H
#define EPARA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct epara_ctx epara_ctx;

/* Task categories (Section 3.1, "Task categories"): sensitivity (latency / frequency) x
 * resource need (<1 GPU / >1 GPU).  The >1 GPU categories need model parallelism and are
 * rejected by epara_submit with EPARA_E_UNSUPPORTED. */
enum {
  EPARA_CAT_LS_LT1 = 0, /* latency-sensitive, fits one GPU: BS + MT */
  EPARA_CAT_FS_LT1 = 1, /* frequency-sensitive, fits one GPU: MF + MT + BS */
  EPARA_CAT_LS_GT1 = 2,
  EPARA_CAT_FS_GT1 = 3
};

/* Status codes.  TIMEOUT and RESOURCE are two of the request handler's answers
 * (Section 3.2: "timeout", "resource insufficiency"). */
enum {
  EPARA_OK = 0,
  EPARA_PENDING = 1,
  EPARA_E_INVALID = -1,
  EPARA_E_UNSUPPORTED = -2,
  EPARA_E_TIMEOUT = -3,
  EPARA_E_RESOURCE = -4,
  EPARA_E_DEVICE = -5,
  EPARA_E_CUDA = -6
};

enum { EPARA_MODEL_MLP = 0, EPARA_MODEL_VIT = 1, EPARA_MODEL_DECODER = 2 };

/* EPARA_GEMM_TCGEN05: the tensor-core kernels, with an encoder's MLP block (FC1, GELU, FC2, residual) run as one
 * fused kernel where its shapes allow (d a multiple of 64 up to 384, hidden width a multiple of 128, more than
 * 128 rows at capacity).  EPARA_GEMM_TCGEN05_UNFUSED: the same kernels, every GEMM its own launch.  Both round
 * at the same points and reduce in the same order.  EPARA_GEMM_SIMT: plain CUDA-core comparator. */
enum { EPARA_GEMM_TCGEN05 = 0, EPARA_GEMM_SIMT = 1, EPARA_GEMM_TCGEN05_UNFUSED = 2 };

#define EPARA_KV_PAGE 16 /* tokens per KV page */

typedef struct {
  int device;             /* CUDA device ordinal; made current by every call */
  void* workspace;        /* device, caller-owned scratch for activations and descriptors */
  size_t workspace_bytes;
  int cap_ls;             /* BS cap of a latency-sensitive group per model per step (0 -> 4) */
  int cap_fs;             /* BS cap of a frequency-sensitive group (0 -> 256) */
  int mf_max;             /* MF: max inter-frame count per stream; 0 = plain oldest-first batching */
  int gemm_impl;          /* EPARA_GEMM_TCGEN05 (default), EPARA_GEMM_TCGEN05_UNFUSED or EPARA_GEMM_SIMT */
  int max_queue;          /* queued requests per (model, category) before RESOURCE (0 -> 4096) */
  int profile;            /* 1: bracket every launch with CUDA events (see epara_step_profile) */
} epara_config;

/* Model description.  `tensors` is a host array of device pointers to bf16 tensors in this order:
 *  MLP     : W_0 [dims[1], dims[0]], b_0 [dims[1]], W_1, b_1, ...          (GELU between layers,
 *            none after the last)
 *  VIT     : W_pe [d, 3*patch*patch], b_pe [d], cls [d], pos [T, d], then per layer
 *            ln1_g, ln1_b, Wqkv [3d, d] (rows q;k;v), bqkv, Wo [d,d], bo, ln2_g, ln2_b,
 *            W1 [ffn, d], b1, W2 [d, ffn], b2, then lnf_g, lnf_b, Whead [vocab, d], bhead.
 *            T = (img/patch)^2 + 1; pre-LN encoder, LayerNorm eps 1e-6, exact-erf GELU.
 *  DECODER : Emb [vocab, d], then per layer g1 [d], Wqkv [(Hq+2Hkv)*hd, d] (rows q;k;v),
 *            Wo [d, Hq*hd], g2 [d], Wgu [2*ffn, d] (row 2j = gate j, row 2j+1 = up j),
 *            Wd [d, ffn], then gf [d], Wlm [vocab, d].  RMSNorm eps 1e-5, interleaved-pair
 *            RoPE base 10000, SwiGLU.
 * Every weight matrix is [out_features, in_features] with in_features contiguous and a
 * multiple of 8.  kv_pool (decoder): bf16 [n_layers][kv_pages][2 (K,V)][Hkv][16][hd]. */
typedef struct {
  int kind;
  int n_layers;
  int d;
  int n_heads;      /* query heads */
  int n_kv_heads;   /* decoder only */
  int head_dim;
  int ffn;
  int vocab;        /* decoder vocabulary / ViT class count / ignored for MLP */
  int img, patch;   /* ViT only */
  const int* mlp_dims;          /* host, n_layers + 1 entries, MLP only */
  const void* const* tensors;   /* host array of device pointers */
  int n_tensors;
  void* kv_pool;                /* device, decoder only */
  long long kv_pages;
  int max_kv_len;               /* decoder: longest cached length a request may have */
  int max_batch;                /* rows reserved in the workspace (0 -> cap_ls + cap_fs): the most requests of a step;
                                   for a decoder the most TOKENS of a step (a decode request is one, a prompt chunk
                                   of n tokens is n); requests beyond it wait for the next step */
  void* trace;                  /* device, decoder only, may be NULL: when given, every step copies the model's
                                   residual stream into it after the embedding and after each layer, fp32
                                   [n_layers + 1][max_batch][d] (row = the request's place in its batch).  For
                                   checking the layers one by one; costs n_layers + 1 small copies per step. */
} epara_model_desc;

/* One request.  Unused fields are ignored for the model's kind. */
typedef struct {
  const void* input;        /* device: MLP bf16 [dims[0]]; VIT bf16 [3, img, img]; DECODER: NULL */
  int token;                /* decoder: id of the token being decoded */
  int kv_len;               /* decoder: cached tokens L; the new token is written at slot L and
                               attention runs over L + 1 tokens */
  const int32_t* block_table; /* device int32 [n_blocks], page ids; needs n_blocks >= (L + n - 1)/16 + 1 */
  int n_blocks;
  const int32_t* tokens;    /* decoder, HOST, read during epara_submit only: with n_tokens = n > 1 the request is a
                               prompt chunk (the prefill phase of an LLM request, Section 4.3): token t goes to
                               position L + t, its k, v are appended there, and it attends causally to positions
                               0 .. L + t.  L = 0 is a whole prompt, L > 0 a later chunk of a chunked prefill.
                               The outputs are the LAST token's logits and argmax.  A chunk takes n of the model's
                               max_batch rows and may share its step with decode requests.  Head sizes 64 and 128. */
  int n_tokens;             /* 0 or 1: a decode request of `token` (or tokens[0] when given) */
  long long deadline_ns;    /* absolute time after which the request is dropped; 0 = none */
  long long arrival_ns;
  int stream;               /* frequency-sensitive stream id (MF groups frames per stream) */
  void* out_logits;         /* device bf16 [n_out] (MLP: last width; VIT/DECODER: vocab) */
  int32_t* out_argmax;      /* device int32 [1]; lowest index wins ties; may be NULL */
} epara_inputs;

typedef struct {
  uint64_t step_id;
  int admitted[2];          /* per category */
  int dropped[2];           /* timed out at admission */
  int launches;             /* kernels launched by this step */
  int gemm_groups;
  double gemm_flops;        /* 2 M N K over all GEMM groups */
  double weight_bytes;      /* bytes of weight matrices the step streams */
  double kv_bytes;          /* bytes of cached K/V the step reads */
  double stream_gemm_flops;   /* the part of gemm_flops in weight-streaming launches (groups of at most 16 rows) */
  double stream_weight_bytes; /* the part of weight_bytes in those launches */
  int prefill_tokens;         /* tokens of the step's prompt chunks */
} epara_step_info;

typedef struct {
  int status;               /* EPARA_OK, EPARA_E_TIMEOUT (dropped), EPARA_E_DEVICE, EPARA_E_CUDA, EPARA_E_RESOURCE */
  uint64_t step_id;
  void* logits;             /* the request's out_logits */
  int n_out;
  int32_t* argmax;
  int device_error;         /* with EPARA_E_DEVICE: the code a kernel of the step left in the step's status word.
                               1..49: a bounded wait ran out (which role gave up); 101: a block table named a page
                               outside the model's kv_pages at the append; 102: the same at an attention read.
                               The accesses behind 101 / 102 are skipped, never performed. */
} epara_output;

/* Kinds of kernels a step launches (index into epara_step_profile arrays). */
enum {
  EPARA_K_GATHER = 0, EPARA_K_NORM = 1, EPARA_K_GEMM = 2, EPARA_K_ROPE = 3, EPARA_K_ATTN_DEC = 4,
  EPARA_K_ATTN_COMBINE = 5, EPARA_K_ATTN_ENC = 6, EPARA_K_ASSEMBLE = 7, EPARA_K_OUTPUT = 8,
  EPARA_K_GEMM_STREAM = 9,  /* the weight-streaming GEMM launches (groups of at most 16 rows); EPARA_K_GEMM holds
                               the tensor-core launches */
  EPARA_K_TRACE = 10,       /* copies into epara_model_desc.trace */
  EPARA_K_ATTN_PREFILL = 11, /* causal attention of prompt chunks */
  EPARA_K_COUNT = 12
};

/* Creates a context on cfg->device.  Returns INVALID (null/unaligned workspace), CUDA. */
int epara_init(const epara_config* cfg, epara_ctx** out);

/* "Placement" of a service on this GPU (the paper pre-places models because loading is slow,
 * Section 3.3): records the pointers, reserves activation workspace for max_batch rows and
 * builds the TMA tensor maps.  RESOURCE if the workspace is too small, INVALID on bad dims. */
int epara_register_model(epara_ctx*, const epara_model_desc* m, int* model_id);

/* Queues one request (host only, no device work).  UNSUPPORTED for the >1 GPU categories,
 * INVALID for bad ids/pointers/lengths, RESOURCE when the queue is full. */
int epara_submit(epara_ctx*, int model_id, int category, const epara_inputs* in, uint64_t* ticket);

/* n requests of one (model, category) in one call, in order; same checks as epara_submit.  Stops at
 * the first rejected request: *n_accepted (may be NULL) counts those queued, tickets[i] is filled
 * for each of them, and the status of the rejected one is returned. */
int epara_submit_many(epara_ctx*, int model_id, int category, const epara_inputs* in, int n, uint64_t* tickets,
                      int* n_accepted);

/* Runs one step on `cuda_stream` (a cudaStream_t), asynchronously:
 *  - drops requests whose deadline_ns < now_ns (Section 3.2, first handler rule);
 *  - per model admits the oldest <= cap_ls latency-sensitive requests, then frequency-
 *    sensitive ones up to cap_fs, by MF when mf_max > 0: floor(cap_fs / mf_max) streams
 *    (Eq. 5), the same number of frames from each;
 *  - runs all admitted groups of all models together, one grouped launch per kernel kind
 *    per dependency wave.
 * now_ns < 0 uses the host's monotonic clock.  info may be NULL. */
int epara_step(epara_ctx*, void* cuda_stream, long long now_ns, epara_step_info* info);

/* PENDING until the step that took the ticket has finished on the device (never blocks); then the
 * request's final answer, also in out->status: OK with out filled; TIMEOUT if the request was dropped at
 * admission; DEVICE when a kernel of its step reported an error (out->device_error has the code; every
 * request of that step answers DEVICE, and the step's outputs must not be used); CUDA or RESOURCE when
 * its step failed on the host after admission (a failed copy or launch, descriptors that did not fit):
 * such requests are not re-queued.  Every step has a status word of its own, so a device error marks one
 * step only.  INVALID for an unknown (or already collected) ticket.  A ticket still queued is PENDING.
 * An answer stays available until it is collected, however many steps run in between. */
int epara_collect(epara_ctx*, uint64_t ticket, epara_output* out);

/* With cfg.profile = 1: per kernel kind, total milliseconds and launch count of the most
 * recent finished step (arrays of EPARA_K_COUNT).  Synchronises that step.  */
int epara_step_profile(epara_ctx*, float* ms_per_kind, int* launches_per_kind);

/* Switches the per-launch event bracketing of epara_config.profile on (1) or off (0). */
int epara_set_profile(epara_ctx*, int on);
/* Most launches a profiled step may have (default 4096); a profiled step with more answers RESOURCE and
 * runs nothing, its requests answer RESOURCE at collect. */
int epara_set_max_profile_launches(epara_ctx*, int n);

int epara_destroy(epara_ctx*);
const char* epara_strerror(int status);

/* Bytes of workspace epara_register_model will reserve for this model under cfg. */
size_t epara_model_workspace_bytes(const epara_config* cfg, const epara_model_desc* m);

/* ---- host policy, exposed for testing and for callers that plan ahead (pure host code) ---- */

/* Eq. 4: DP group count = ceil(required frame rate / frame rate of one group). */
int epara_dp_group_count(double required_fps, double group_fps);
/* Eq. 5: inter-request count = floor(BS / max inter-frame count). */
int epara_inter_request_count(int bs, int mf_max);
/* Admission of one queue (the rule epara_step applies).  Arrays are host memory of n entries in
 * arrival order; out_admitted/out_dropped need room for n entries.  Returns EPARA_OK. */
int epara_admit_queue(int n, const uint64_t* tickets, const long long* deadline_ns, const int* streams,
                      long long now_ns, int cap, int mf_max,
                      uint64_t* out_admitted, int* n_admitted, uint64_t* out_dropped, int* n_dropped);

/* ---- host policies around the step (pure host code): request handling, placement, simulation ----
 *
 * Model.  Servers n = 0 .. n_servers-1 with gpus[n] identical GPUs; a GPU has compute capacity 1 (a service's MPS
 * share `a` is a fraction of it) and `vram` GB.  Server index n_servers is the hypothetical server of Algorithm 1,
 * stage 3: it owns no GPU and places an instance on free GPUs of any real servers.  A placement (service, server)
 * is one instance; it takes n_gpus GPUs, first fit in (server, gpu) order, `a` and `b` on each.
 * A service has a category (0 latency-, 1 frequency-sensitive), a batch size, a latency SLO per request or
 * frame, for frequency-sensitive services the frame rate and the frames of a request (its frames arrive
 * 1 / fps apart), and the profiled compute time c_ms[k] of a batch of up to 2^k requests (the c_ln table of
 * Section 3.3, measured by the offline profiler of Section 4.1).
 * A request reaches `server` at t_ms; u[] are pre-drawn uniform numbers in [0, 1), one per offloading decision. */
#define EPARA_PROFILE_POINTS 10       /* batch sizes 2^0 .. 2^9 (Section 4.1) */
#define EPARA_MAX_OFFLOAD_DRAWS 5     /* the default maximum offloading count (Section 4.1, Table 4) */
typedef struct { int n_servers; const int* gpus; double vram; double sync_ms; double offload_ms; } epara_cluster;
typedef struct {
  double a, b;              /* compute share of a GPU, VRAM in GB, per GPU of an instance */
  int n_gpus;               /* GPUs one instance spans (1 for the "<1 GPU" categories) */
  int cat;                  /* 0 latency-sensitive, 1 frequency-sensitive */
  int bs;                   /* batch size */
  double slo_ms;            /* latency SLO of a request (or of one frame) */
  double fps;               /* frequency-sensitive: required frame rate */
  int frames;               /* frequency-sensitive: frames of one request */
  double c_ms[EPARA_PROFILE_POINTS];
} epara_service;
typedef struct { double t_ms; int service; int server; double u[EPARA_MAX_OFFLOAD_DRAWS]; } epara_request;
typedef struct { int service; int server; } epara_placement;
typedef struct {
  double phi;               /* Eq. 2: satisfied requests; a frequency-sensitive request of F frames counts
                               F x achieved / required frame rate (Section 3.3), at most the frames in time */
  int served, timeout, offload_exceed, insufficient, late, offloads, instances;   /* per work item (request or frame) */
} epara_sim_result;

/* Eq. 1: candidate m has idle goodput p_hat[m] - p_act[m] (theoretical minus actual goodput; negative counts
 * as 0) and is excluded when queued_ms[m] > t_sync_ms[m] + slo_ms; prob[m] = idle / sum of idle (all 0 when no
 * candidate has idle goodput).  All arrays host, n entries. */
int epara_offload_probabilities(int n, const double* p_hat, const double* p_act, const double* queued_ms,
                                const double* t_sync_ms, double slo_ms, double* prob);

/* Event-driven replay (Section 5.2: request scheduling is executed in full, compute latency comes from the
 * lookup tables, a hop costs offload_ms) of the requests against the placements under the request handler's
 * decision list (Section 3.2): an item past its deadline answers timeout; else a local instance that would
 * finish it in time takes it (the server's own first, then the hypothetical server's); else, with max_offload
 * offloads behind it, offloading exceed; else it moves to a server not yet on its path picked by Eq. 1
 * (p_hat: sum of bs / c(bs) over the server's instances of the service; p_act: their completions in
 * [now - 2 sync_ms, now - sync_ms] per second; queued time: the least over those instances), or answers
 * resource insufficiency when no candidate has idle goodput.  An instance runs one batch at a time: the oldest
 * bs items still in time, for c(batch).  Placements that do not fit are skipped.  All pointers host. */
int epara_simulate(const epara_cluster* c, const epara_service* services, int n_services, const epara_request* requests,
                   int n_requests, const epara_placement* placements, int n_placements, int max_offload,
                   epara_sim_result* out);

/* Algorithm 1 (state-aware service placement) over Algorithm 2 (submodular placement for full models), with
 * epara_simulate's phi as the objective: stage 1 places from the priority list (each entry at most once, the
 * loop goes on while phi does not decrease), stage 2 from the set of all (service, real server) pairs, stage 3
 * from the set of all (service, hypothetical server) pairs (both while phi strictly grows).  In every round the
 * candidates that still fit are evaluated, the best ones form the tie set, and its first member in candidate
 * order is placed.  out receives at most out_cap placements in placement order, *n_out their number
 * (RESOURCE when out_cap is too small). */
int epara_place_sssp(const epara_cluster* c, const epara_service* services, int n_services, const epara_request* requests,
                     int n_requests, const epara_placement* priority, int n_priority, int max_offload,
                     epara_placement* out, int out_cap, int* n_out);

/* ---- single-kernel entry points (the same kernels a step launches), for parity tests and
 *      roofline measurement.  All pointers device unless named host. ---- */

typedef struct {
  const void* A;      /* bf16 [M, lda]  */
  const void* W;      /* bf16 [N, ldw], K contiguous */
  void* C;            /* bf16 [M, ldc] (or fp32 when EPARA_EPI_RESID_F32); SwiGLU: [M, N/2].  Pad columns
                         between N and the next multiple of 8 may be overwritten. */
  const void* bias;   /* bf16 [N] or NULL */
  int M, N, K;
  int lda, ldw, ldc;  /* elements; multiples of 8 */
  int epilogue;       /* EPARA_EPI_* flags */
} epara_gemm_problem;

enum { EPARA_EPI_BIAS = 1, EPARA_EPI_GELU = 2, EPARA_EPI_SWIGLU = 4, EPARA_EPI_RESID_F32 = 8 };

/* C_g = epilogue(A_g W_g^T + bias_g) for every problem in one grouped launch.  RESID_F32:
 * C is fp32 and is updated in place, C += A W^T + bias.  `problems` is host memory;
 * `scratch` is device memory, 256-byte aligned, of at least epara_gemm_scratch_bytes_for(device, problems, n)
 * bytes (descriptors, plus fp32 partials for small-M problems that are split along K);
 * epara_gemm_scratch_bytes(n) suffices for EPARA_GEMM_SIMT. */
int epara_grouped_gemm(int device, void* cuda_stream, int impl, const epara_gemm_problem* problems, int n,
                       void* scratch, size_t scratch_bytes);
size_t epara_gemm_scratch_bytes(int n_problems);
size_t epara_gemm_scratch_bytes_for(int device, const epara_gemm_problem* problems, int n);

/* Split-KV paged decode attention with GQA (one layer).  q: bf16 [B, q_stride] (head h at
 * column h*hd); kv_layer: bf16 [kv_pages][2][Hkv][16][hd]; kv_lens int32 [B] = tokens to attend
 * (cached + appended; values outside [0, max_len] are clamped, a request of length 0 leaves its output
 * row unwritten); tables: int32 [B, table_stride]; out bf16 [B, Hq*hd];
 * scratch: at least epara_decode_attention_scratch_bytes(B, Hq, hd, max_len) bytes (descriptor, request
 * table, fp32 chunk partials, chunk counters; the call clears what must start at zero itself).
 * A page id outside [0, kv_pages) is never dereferenced: the page is read as absent and the int32 at byte
 * EPARA_DECODE_STATUS_OFFSET of `scratch` is set to 102 (it is 0 after a clean call). */
#define EPARA_DECODE_STATUS_OFFSET 192
int epara_decode_attention(int device, void* cuda_stream, const void* q, int q_stride, const void* kv_layer,
                           long long kv_pages, const int32_t* kv_lens, const int32_t* tables, int table_stride,
                           void* out, int B, int Hq, int Hkv, int hd, int max_len, void* scratch, size_t scratch_bytes);
size_t epara_decode_attention_scratch_bytes(int B, int Hq, int hd, int max_len);

/* Decode attention for callers that cannot allocate device memory.  (The paper has no counterpart
 * of this call; it exists for how this library gets embedded.)
 *
 * Some users of this library run where cudaMalloc is off limits: a serving process whose framework
 * took the whole device for its own memory pool at start-up, so that a driver allocation now fails
 * or forces the pool to shrink; or a latency-critical loop in which the implicit device-wide
 * synchronisation of cudaMalloc/cudaFree would stall every stream.  Such callers cannot provide the
 * scratch buffer epara_decode_attention asks for.  This variant takes the same inputs and outputs
 * and keeps its scratch (request table and split-KV partials) in an array that is part of the
 * library image: EPARA_STATIC_SCRATCH_BYTES of device memory on every GPU that loads the library,
 * held until the process exits.  It calls no cudaMalloc, cudaFree or any allocating routine.
 *
 * Same kernels, same results as epara_decode_attention.  Arguments as there, minus scratch.
 * Returns EPARA_E_RESOURCE when 256 + roundup256(16 B) + roundup256(B*Hq*ceil(max_len/256)*(hd+2)*4) +
 * 4*B*Hq bytes exceed EPARA_STATIC_SCRATCH_BYTES (nothing is launched), INVALID / UNSUPPORTED / CUDA as
 * the other entry.
 *
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress) and caches
 * it; make that first call outside any stream capture.  All calls on a device share the one array,
 * which keeps whatever the previous call left in it: the request table and the partials are written
 * before they are read, and the per-(request, kv head) chunk counters, the one part that must start
 * at zero, are cleared on the stream by every call (a small set-up kernel, which also writes the call's
 * descriptor from its own arguments, so no host buffer has to outlive the call).  Two calls whose kernels
 * may overlap on the GPU -- different streams without an ordering between them -- race on that array;
 * order them.  epara_decode_attention_static_status copies the last call's status word back (it waits
 * for the device): OK and *code = 0 after a clean call, DEVICE and *code = 102 when a block table named
 * a page outside [0, kv_pages). */
#define EPARA_STATIC_SCRATCH_BYTES (8u << 20)
int epara_decode_attention_static(int device, void* cuda_stream, const void* q, int q_stride, const void* kv_layer,
                                  long long kv_pages, const int32_t* kv_lens, const int32_t* tables, int table_stride,
                                  void* out, int B, int Hq, int Hkv, int hd, int max_len);
int epara_decode_attention_static_status(int device, int* code);
size_t epara_static_scratch_bytes(void);

/* Self-test of the bounded waits (the paper has no counterpart; it exists so that the give-up path of the
 * kernels' waits can be run without making a real kernel misbehave).  Launches one thread that waits, for
 * at most limit_ns (<= 1 s), on a barrier nothing ever arrives at, then synchronises the stream.  Expected
 * answer: EPARA_E_DEVICE with *code = 90 (the wait ran out and the kernel returned by itself).
 * status_dev: device int32 used as the status word; code: host. */
int epara_selftest_bounded_wait(int device, void* cuda_stream, unsigned long long limit_ns, int* status_dev, int* code);

#ifdef __cplusplus
}
#endif
#endif /* EPARA_H */
