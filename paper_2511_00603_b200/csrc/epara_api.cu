// C ABI, category table, admission and step planner (host code).
//
// epara_register_model turns a model into a static list of ops (gather, norm, GEMM, RoPE+append,
// attention, ...) over buffers carved from the caller's workspace, with the TMA maps of every
// GEMM operand built once.  epara_step admits requests per (model, category), then walks all
// active models' op lists together: in each sweep over the kernel kinds, every model whose next
// op is of that kind contributes one group to a single grouped launch (MT: different services in
// one launch; BS: a group's M is its batch).  All descriptors of the step travel in one pinned
// blob with one host-to-device copy.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <chrono>
#include <cmath>
#include <cstring>
#include <deque>
#include <new>
#include <unordered_map>
#include <vector>

#include "../../include/epara.h"
#include "desc.h"
#include "kernels.h"

using namespace epara;

namespace {

constexpr int N_SLOTS = 4;
constexpr size_t BLOB_BYTES = 4u << 20;
constexpr int MAX_PROFILE_LAUNCHES = 4096;

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int round_up(int v, int a) { return (v + a - 1) / a * a; }

// ---- TMA map encoding through the runtime's driver entry point (no link against libcuda) ----
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

// bf16 matrix [rows, cols] with leading dimension ld, cols innermost; box = 64 cols x box_rows,
// 128-byte swizzle, out-of-range elements read as zero.
bool make_tmap(CUtensorMap* tm, const void* ptr, long long rows, long long cols, long long ld, int box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Output map of a GEMM for the epilogue's TMA stores: rows of 64 bytes (SwiGLU: 32 bytes) per box row,
// matching swizzle, 32 rows per box.
bool make_tmap_c(CUtensorMap* tm, void* C, long long rows, int N, int ldc, int epi) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  const bool f32 = (epi & EPI_RESID_F32) != 0, swi = (epi & EPI_SWIGLU) != 0;
  const int cols = swi ? N / 2 : N;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ldc * (f32 ? 4 : 2)};
  cuuint32_t box[2] = {(cuuint32_t)(f32 ? 16 : (swi ? 16 : 32)), 32};
  cuuint32_t estr[2] = {1, 1};
  return fn(tm, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, C, dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swi ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_64B,
            CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct Op {
  int kind;           // EPARA_K_*
  int rows_per_req;   // rows of this op = batch * rows_per_req ...
  int per_token;      // ... or, for a decoder's token-wise ops, the step's token rows (a prompt chunk has several)
  int last_rows;      // norm: output row b reads the last token row of request b
  AttnPrefillGroup apre;
  GemmGroup gemm;
  MlpGroup mlp;          // EPARA_K_GEMM with gemm.stream == 4: FC1, GELU, FC2 and the residual update in one kernel
  NormGroup norm;
  GatherGroup gather;
  RopeGroup rope;
  AttnDecGroup adec;
  AttnEncGroup aenc;
  AssembleGroup asmb;
  OutputGroup outp;
  double weight_bytes;
  const void* trace_src;   // EPARA_K_TRACE: copy rows * trace_row_bytes from here ...
  void* trace_dst;         // ... to here
  size_t trace_row_bytes;
};

struct Request {
  uint64_t ticket;
  epara_inputs in;
  std::vector<int32_t> toks;   // decoder prompt chunk (n_tokens > 1): a copy of the caller's token ids
  int n_tok() const { return toks.empty() ? 1 : (int)toks.size(); }
};

// T_INFLIGHT: admitted to a step whose slot still holds the step's record.  T_DONE: the final answer is
// in `result` (a dropped request, a step that failed on the host, or a step whose slot was recycled).
enum { T_QUEUED = 0, T_INFLIGHT = 1, T_DONE = 2 };
struct Ticket {
  int state;
  int model;
  uint64_t step;
  void* out_logits;
  int32_t* out_argmax;
  int result;          // T_DONE: EPARA_OK / EPARA_E_TIMEOUT / EPARA_E_DEVICE / EPARA_E_CUDA / EPARA_E_RESOURCE
  int device_error;    // T_DONE with EPARA_E_DEVICE: the code the kernel recorded
};

struct Model {
  epara_model_desc d;
  std::vector<const void*> tensors;
  std::vector<int> dims;
  int max_batch;
  int n_out;
  std::vector<Op> ops;
  std::deque<Request> q[2];
  int max_chunks;       // decoder
  double kv_bytes_per_token;
  size_t splitk_bytes = 0, splitk_tiles = 0;   // largest split-k partial buffer / tile count of its GEMMs
};

// The first BLOB_HEADER bytes of a slot's device blob hold the step's status word; the upload of the blob
// writes zeros there, so every step starts with a clear word of its own.
constexpr size_t BLOB_HEADER = 64;
struct Slot {
  unsigned char* host;  // pinned blob
  unsigned char* dev;   // device blob (in the workspace)
  int* status_host;     // pinned copy of the step's status word, valid once `done` has fired
  cudaEvent_t done;
  uint64_t step_id;     // 0 = never used
  bool busy;
  bool profiled;        // the step in this slot was bracketed with events
  int launch_status;    // EPARA_OK, or what a failed launch of the step maps to
  std::vector<uint64_t> tickets;   // requests admitted to the step in this slot
  std::vector<cudaEvent_t> prof;   // 2 per launch when profiling
  std::vector<int> prof_kind;
};

struct Launch {
  int kind;
  size_t off;
  int n_groups;
  int p0, p1, p2, p3;
  const void* src;   // EPARA_K_TRACE
  void* dst;
  size_t bytes;
};

}  // namespace

struct epara_ctx {
  epara_config cfg;
  int sm_count;
  unsigned char* ws;
  size_t ws_bytes, ws_used;
  std::vector<Model*> models;
  std::unordered_map<uint64_t, Ticket> tickets;
  uint64_t next_ticket, next_step;
  Slot slots[N_SLOTS];
  uint64_t last_step_slot;
  int max_profile_launches;
};

namespace {

void* carve(epara_ctx* c, size_t bytes) {
  const size_t off = align_up(c->ws_used, 256);
  if (off + bytes > c->ws_bytes) return nullptr;
  c->ws_used = off + bytes;
  return c->ws + off;
}

size_t carve_size(size_t& used, size_t bytes) {
  const size_t off = align_up(used, 256);
  used = off + bytes;
  return off;
}

// SM count of a device (cached; 148 on a B200).  Tile widths of the weight-streaming GEMMs depend on it.
int device_sm_count(int device) {
  static int cache[64] = {0};
  if (device < 0 || device >= 64) return 148;
  if (cache[device] == 0) {
    int sm = 0;
    if (cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sm <= 0) return 148;
    cache[device] = sm;
  }
  return cache[device];
}

// Builds the op list of a model.  With c == nullptr only counts workspace bytes (in *need).
// Buffers are requested through `get`, which either carves or counts.
struct Builder {
  epara_ctx* c;
  size_t need;
  bool fail;
  int sm_count;
  int gemm_impl;
  void* get(size_t bytes) {
    if (!c) { carve_size(need, bytes); return reinterpret_cast<void*>(size_t(256)); }
    void* p = carve(c, bytes);
    if (!p) fail = true;
    return p;
  }
};

bool add_gemm(Builder& bl, Model* m, const void* A, int lda, long long rows_cap, const void* W, int N, int K,
              void* C, int ldc, const void* bias, int epi, int rows_per_req) {
  const int sm_count = bl.sm_count;
  const long long max_rows = (long long)m->max_batch * rows_per_req;   // the most rows this op ever sees
  Op op;
  memset(&op, 0, sizeof(op));
  op.kind = EPARA_K_GEMM;
  op.rows_per_req = rows_per_req;
  GemmGroup& g = op.gemm;
  g.A = (const bf16*)A; g.W = (const bf16*)W; g.C = C; g.bias = (const bf16*)bias;
  g.N = N; g.K = K; g.lda = lda; g.ldw = K; g.ldc = ldc; g.epi = epi | (bias ? EPI_BIAS : 0);
  op.weight_bytes = 2.0 * N * K;
  gemm_tc_config(rows_cap, N, K, g.epi, sm_count, &g.bn, &g.ksplit);
  if (max_rows <= GEMM_STREAM_MAX_ROWS && bl.gemm_impl != EPARA_GEMM_SIMT) {
    g.stream = 1; g.bn = 16; g.ksplit = 1;
  } else if (max_rows <= GEMM_SWAP_MAX_ROWS && bl.gemm_impl != EPARA_GEMM_SIMT) {
    g.stream = 3;                              // W as the MMA's 128-row operand, the batch as its N
    g.bn = round_up((int)max_rows, 16);
    g.ksplit = gemm_swap_ksplit(N, K, sm_count);
  } else if (bl.gemm_impl != EPARA_GEMM_SIMT && gemm_tc_pair_eligible(rows_cap, N, K, g.epi, g.bn, g.ksplit)) {
    g.stream = 2;                              // 256-row tiles on CTA pairs
  }
  if (g.ksplit > 1 && g.stream == 0) {
    const size_t tiles_m = (size_t)((rows_cap + TC_BM - 1) / TC_BM), tiles_n = (size_t)((N + g.bn - 1) / g.bn);
    m->splitk_bytes = std::max(m->splitk_bytes, (size_t)g.ksplit * tiles_m * TC_BM * tiles_n * g.bn * 4);
    m->splitk_tiles = std::max(m->splitk_tiles, tiles_m * tiles_n);
  }
  if (bl.c && g.stream == 3) {
    if (!make_tmap(&g.tmA, A, rows_cap, K, lda, g.bn)) return false;
    if (!make_tmap(&g.tmW, W, N, K, K, TC_BM)) return false;
  } else if (bl.c && g.stream != 1) {
    if (!make_tmap(&g.tmA, A, rows_cap, K, lda, TC_BM)) return false;
    if (!make_tmap(&g.tmW, W, N, K, K, g.stream == 2 ? g.bn / 2 : g.bn)) return false;   // a pair's CTA loads half of the W rows
    if (!make_tmap_c(&g.tmC, C, rows_cap, N, ldc, g.epi)) return false;
  }
  g.c_rows = (int)rows_cap;
  m->ops.push_back(op);
  return true;
}

// An encoder's MLP block as one fused op (see MlpGroup).  gemm.N / gemm.K carry the shapes for the step's
// flop and byte accounting; gemm.stream == 4 routes the op to the fused kernel's launch.
bool add_mlp(Builder& bl, Model* m, const void* X, long long rows_cap, const void* W1, const void* b1, const void* W2,
             const void* b2, float* Z, int d, int F, int rows_per_req) {
  Op op;
  memset(&op, 0, sizeof(op));
  op.kind = EPARA_K_GEMM;
  op.rows_per_req = rows_per_req;
  op.gemm.stream = 4; op.gemm.N = d; op.gemm.K = F; op.gemm.ksplit = 1; op.gemm.bn = d;
  op.weight_bytes = 2.0 * 2.0 * d * F;
  MlpGroup& g = op.mlp;
  g.b1 = (const bf16*)b1; g.b2 = (const bf16*)b2; g.d = d; g.F = F; g.c_rows = (int)rows_cap;
  if (bl.c) {
    const int n2 = d > 256 ? d / 2 : d;
    if (!make_tmap(&g.tmX, X, rows_cap, d, d, TC_BM)) return false;
    if (!make_tmap(&g.tmW1, W1, F, d, d, 64)) return false;
    if (!make_tmap(&g.tmW2, W2, d, F, F, n2 / 2)) return false;
    if (!make_tmap_c(&g.tmC, Z, rows_cap, d, d, EPI_RESID_F32)) return false;
  }
  m->ops.push_back(op);
  return true;
}

void add_norm(Model* m, const float* x, long long x_stride, bf16* y, const void* gamma, const void* beta, int d,
              int kind, float eps, int rows_per_req) {
  Op op;
  memset(&op, 0, sizeof(op));
  op.kind = EPARA_K_NORM;
  op.rows_per_req = rows_per_req;
  op.norm.x = x; op.norm.y = y; op.norm.gamma = (const bf16*)gamma; op.norm.beta = (const bf16*)beta;
  op.norm.x_stride = x_stride; op.norm.d = d; op.norm.kind = kind; op.norm.eps = eps;
  m->ops.push_back(op);
}

int validate_desc(const epara_model_desc* d) {
  if (!d || !d->tensors) return EPARA_E_INVALID;
  for (int i = 0; i < d->n_tensors; ++i)
    if (!d->tensors[i] || (reinterpret_cast<uintptr_t>(d->tensors[i]) & 15)) return EPARA_E_INVALID;
  if (d->n_layers <= 0) return EPARA_E_INVALID;
  switch (d->kind) {
    case EPARA_MODEL_MLP:
      if (!d->mlp_dims || d->n_tensors != 2 * d->n_layers) return EPARA_E_INVALID;
      for (int i = 0; i < d->n_layers; ++i)
        if (d->mlp_dims[i] <= 0 || d->mlp_dims[i] % 8) return EPARA_E_INVALID;
      if (d->mlp_dims[d->n_layers] <= 0) return EPARA_E_INVALID;
      return EPARA_OK;
    case EPARA_MODEL_VIT:
      if (d->n_tensors != 4 + 12 * d->n_layers + 4) return EPARA_E_INVALID;
      if (d->d <= 0 || d->d % 8 || d->d > 8192 || d->n_heads <= 0 || d->d != d->n_heads * d->head_dim)
        return EPARA_E_INVALID;
      if (d->head_dim != 64) return EPARA_E_UNSUPPORTED;
      if (d->patch <= 0 || d->patch % 8 || d->img <= 0 || d->img % d->patch || d->img % 8) return EPARA_E_INVALID;
      if (d->ffn <= 0 || d->ffn % 8 || d->vocab <= 0) return EPARA_E_INVALID;
      return EPARA_OK;
    case EPARA_MODEL_DECODER: {
      if (d->n_tensors != 1 + 6 * d->n_layers + 2) return EPARA_E_INVALID;
      if (d->d <= 0 || d->d % 8 || d->d > 8192 || d->ffn <= 0 || d->ffn % 8 || d->vocab <= 0) return EPARA_E_INVALID;
      if (d->n_heads <= 0 || d->n_kv_heads <= 0 || d->n_heads % d->n_kv_heads) return EPARA_E_INVALID;
      const int g = d->n_heads / d->n_kv_heads, hd = d->head_dim;
      const bool hd_ok = hd == 16 || hd == 32 || hd == 64 || hd == 128;
      const bool g_ok = g == 1 || g == 2 || g == 4 || (g == 8 && hd >= 64);
      if (!hd_ok || !g_ok) return EPARA_E_UNSUPPORTED;
      if (!d->kv_pool || (reinterpret_cast<uintptr_t>(d->kv_pool) & 15) || d->kv_pages <= 0 || d->max_kv_len < 0)
        return EPARA_E_INVALID;
      return EPARA_OK;
    }
    default:
      return EPARA_E_INVALID;
  }
}

int build_model(Builder& bl, Model* m, const epara_config& cfg) {
  const epara_model_desc& d = m->d;
  const int B = m->max_batch;
  const long long Bcap = round_up(B, TC_BM);
  const void* const* t = m->tensors.data();
  if (d.kind == EPARA_MODEL_MLP) {
    const int L = d.n_layers;
    int maxw = 0;
    for (int i = 1; i <= L; ++i) maxw = std::max(maxw, round_up(m->dims[i], 8));
    bf16* x0 = (bf16*)bl.get((size_t)Bcap * m->dims[0] * 2);
    bf16* pp[2] = {(bf16*)bl.get((size_t)Bcap * maxw * 2), (bf16*)bl.get((size_t)Bcap * maxw * 2)};
    if (bl.fail) return EPARA_E_RESOURCE;
    Op g;
    memset(&g, 0, sizeof(g));
    g.kind = EPARA_K_GATHER; g.rows_per_req = 1;
    g.gather.kind = GATHER_ROWS; g.gather.out = x0; g.gather.width = m->dims[0]; g.gather.ld = m->dims[0];
    m->ops.push_back(g);
    const bf16* in = x0;
    int ld_in = m->dims[0];
    for (int l = 0; l < L; ++l) {
      const int N = m->dims[l + 1], K = m->dims[l], ldc = round_up(N, 8);
      bf16* out = pp[l & 1];
      if (!add_gemm(bl, m, in, ld_in, Bcap, t[2 * l], N, K, out, ldc, t[2 * l + 1], (l + 1 < L) ? EPI_GELU : 0, 1))
        return EPARA_E_CUDA;
      in = out; ld_in = ldc;
    }
    Op o;
    memset(&o, 0, sizeof(o));
    o.kind = EPARA_K_OUTPUT; o.rows_per_req = 1;
    o.outp.logits = in; o.outp.N = m->dims[L]; o.outp.ld = ld_in;
    m->ops.push_back(o);
    m->n_out = m->dims[L];
    return EPARA_OK;
  }
  if (d.kind == EPARA_MODEL_VIT) {
    const int dm = d.d, T = (d.img / d.patch) * (d.img / d.patch) + 1, np = T - 1;
    const int pk = 3 * d.patch * d.patch;
    const long long Mcap = round_up(B * T, TC_BM);
    const int fw = std::max(d.ffn, pk);
    float* z = (float*)bl.get((size_t)Mcap * dm * 4);
    bf16* h = (bf16*)bl.get((size_t)Mcap * dm * 2);
    bf16* qkv = (bf16*)bl.get((size_t)Mcap * 3 * dm * 2);
    bf16* a = (bf16*)bl.get((size_t)Mcap * dm * 2);
    bf16* f = (bf16*)bl.get((size_t)Mcap * fw * 2);
    bf16* cvec = (bf16*)bl.get((size_t)Bcap * dm * 2);
    const int ldl = round_up(d.vocab, 8);
    bf16* logits = (bf16*)bl.get((size_t)Bcap * ldl * 2);
    if (bl.fail) return EPARA_E_RESOURCE;
    Op g;
    memset(&g, 0, sizeof(g));
    g.kind = EPARA_K_GATHER; g.rows_per_req = np;
    g.gather.kind = GATHER_PATCH; g.gather.out = f; g.gather.width = pk; g.gather.ld = pk;
    g.gather.img = d.img; g.gather.patch = d.patch;
    m->ops.push_back(g);
    if (!add_gemm(bl, m, f, pk, Mcap, t[0], dm, pk, a, dm, t[1], 0, np)) return EPARA_E_CUDA;
    Op as;
    memset(&as, 0, sizeof(as));
    as.kind = EPARA_K_ASSEMBLE; as.rows_per_req = T;
    as.asmb.E = a; as.asmb.cls = (const bf16*)t[2]; as.asmb.pos = (const bf16*)t[3]; as.asmb.z = z;
    as.asmb.T = T; as.asmb.d = dm;
    m->ops.push_back(as);
    for (int l = 0; l < d.n_layers; ++l) {
      const void* const* w = t + 4 + 12 * l;
      add_norm(m, z, dm, h, w[0], w[1], dm, NORM_LN, 1e-6f, T);
      if (!add_gemm(bl, m, h, dm, Mcap, w[2], 3 * dm, dm, qkv, 3 * dm, w[3], 0, T)) return EPARA_E_CUDA;
      Op at;
      memset(&at, 0, sizeof(at));
      at.kind = EPARA_K_ATTN_ENC; at.rows_per_req = T;
      at.aenc.qkv = qkv; at.aenc.out = a; at.aenc.T = T; at.aenc.H = d.n_heads; at.aenc.hd = d.head_dim;
      at.aenc.KP = round_up(T, 16);
      at.aenc.tc = (d.head_dim == 64 && T <= ENC_TC_MAX_T && bl.gemm_impl != EPARA_GEMM_SIMT) ? 1 : 0;
      if (at.aenc.tc && bl.c) {
        if (!make_tmap(&at.aenc.tmQ, qkv, Mcap, 3 * dm, 3 * dm, 128)) return EPARA_E_CUDA;
        if (!make_tmap(&at.aenc.tmKV, qkv, Mcap, 3 * dm, 3 * dm, at.aenc.KP)) return EPARA_E_CUDA;
      }
      m->ops.push_back(at);
      if (!add_gemm(bl, m, a, dm, Mcap, w[4], dm, dm, z, dm, w[5], EPI_RESID_F32, T)) return EPARA_E_CUDA;
      add_norm(m, z, dm, h, w[6], w[7], dm, NORM_LN, 1e-6f, T);
      if (bl.gemm_impl == EPARA_GEMM_TCGEN05 && gemm_mlp_eligible(Mcap, dm, d.ffn)) {
        if (!add_mlp(bl, m, h, Mcap, w[8], w[9], w[10], w[11], z, dm, d.ffn, T)) return EPARA_E_CUDA;
      } else {
        if (!add_gemm(bl, m, h, dm, Mcap, w[8], d.ffn, dm, f, d.ffn, w[9], EPI_GELU, T)) return EPARA_E_CUDA;
        if (!add_gemm(bl, m, f, d.ffn, Mcap, w[10], dm, d.ffn, z, dm, w[11], EPI_RESID_F32, T)) return EPARA_E_CUDA;
      }
    }
    const void* const* w = t + 4 + 12 * d.n_layers;
    add_norm(m, z, (long long)T * dm, cvec, w[0], w[1], dm, NORM_LN, 1e-6f, 1);
    if (!add_gemm(bl, m, cvec, dm, Bcap, w[2], d.vocab, dm, logits, ldl, w[3], 0, 1)) return EPARA_E_CUDA;
    Op o;
    memset(&o, 0, sizeof(o));
    o.kind = EPARA_K_OUTPUT; o.rows_per_req = 1;
    o.outp.logits = logits; o.outp.N = d.vocab; o.outp.ld = ldl;
    m->ops.push_back(o);
    m->n_out = d.vocab;
    return EPARA_OK;
  }
  // decoder
  const int dm = d.d, Hq = d.n_heads, Hkv = d.n_kv_heads, hd = d.head_dim, F = d.ffn;
  const int nq = (Hq + 2 * Hkv) * hd;
  m->max_chunks = (d.max_kv_len + 1 + ATTN_CHUNK - 1) / ATTN_CHUNK;
  m->kv_bytes_per_token = 2.0 * Hkv * hd * 2.0 * d.n_layers;
  float* x = (float*)bl.get((size_t)Bcap * dm * 4);
  bf16* h = (bf16*)bl.get((size_t)Bcap * dm * 2);
  bf16* qkv = (bf16*)bl.get((size_t)Bcap * nq * 2);
  bf16* a = (bf16*)bl.get((size_t)Bcap * Hq * hd * 2);
  bf16* f = (bf16*)bl.get((size_t)Bcap * F * 2);
  const int ldl = round_up(d.vocab, 8);
  bf16* logits = (bf16*)bl.get((size_t)Bcap * ldl * 2);
  float* partial = (float*)bl.get((size_t)B * Hq * m->max_chunks * (hd + 2) * 4);
  int* chunk_counters = (int*)bl.get((size_t)B * Hkv * sizeof(int));
  float2* rope_cs = (float2*)bl.get((size_t)(d.max_kv_len + 1) * (hd / 2) * sizeof(float2));
  if (bl.fail) return EPARA_E_RESOURCE;
  if (bl.c) {
    // rotation table: angles in fp64 on the host, (cos, sin) rounded once to fp32
    const int half = hd / 2;
    std::vector<double> inv_freq(half);
    for (int j = 0; j < half; ++j) inv_freq[j] = std::pow(10000.0, -2.0 * j / hd);
    std::vector<float2> cs((size_t)(d.max_kv_len + 1) * half);
    for (int p = 0; p <= d.max_kv_len; ++p)
      for (int j = 0; j < half; ++j) {
        const double ang = (double)p * inv_freq[j];
        cs[(size_t)p * half + j] = make_float2((float)std::cos(ang), (float)std::sin(ang));
      }
    if (cudaMemcpy(rope_cs, cs.data(), cs.size() * sizeof(float2), cudaMemcpyHostToDevice) != cudaSuccess) return EPARA_E_CUDA;
    if (cudaMemset(chunk_counters, 0, (size_t)B * Hkv * sizeof(int)) != cudaSuccess) return EPARA_E_CUDA;
  }
  Op g;
  memset(&g, 0, sizeof(g));
  g.kind = EPARA_K_GATHER; g.rows_per_req = 1;
  g.gather.kind = GATHER_EMB; g.gather.out = x; g.gather.emb = (const bf16*)t[0]; g.gather.width = dm; g.gather.ld = dm;
  m->ops.push_back(g);
  // debug trace: the residual stream after the embedding and after every layer, [n_layers + 1][max_batch][d] fp32
  auto add_trace = [&](int index) {
    if (!d.trace) return;
    Op tr;
    memset(&tr, 0, sizeof(tr));
    tr.kind = EPARA_K_TRACE; tr.rows_per_req = 1;
    tr.trace_src = x; tr.trace_dst = (float*)d.trace + (size_t)index * B * dm; tr.trace_row_bytes = (size_t)dm * 4;
    m->ops.push_back(tr);
  };
  add_trace(0);
  const size_t layer_elems = (size_t)d.kv_pages * 2 * Hkv * 16 * hd;
  for (int l = 0; l < d.n_layers; ++l) {
    const void* const* w = t + 1 + 6 * l;
    bf16* kv_layer = (bf16*)d.kv_pool + layer_elems * l;
    add_norm(m, x, dm, h, w[0], nullptr, dm, NORM_RMS, 1e-5f, 1);
    if (!add_gemm(bl, m, h, dm, Bcap, w[1], nq, dm, qkv, nq, nullptr, 0, 1)) return EPARA_E_CUDA;
    Op r;
    memset(&r, 0, sizeof(r));
    r.kind = EPARA_K_ROPE; r.rows_per_req = 1;
    r.rope.qkv = qkv; r.rope.kv_layer = kv_layer; r.rope.cs = rope_cs;
    r.rope.Hq = Hq; r.rope.Hkv = Hkv; r.rope.hd = hd; r.rope.kv_pages = d.kv_pages;
    m->ops.push_back(r);
    Op at;
    memset(&at, 0, sizeof(at));
    at.kind = EPARA_K_ATTN_DEC; at.rows_per_req = 1;
    at.adec.q = qkv; at.adec.q_stride = nq; at.adec.kv_layer = kv_layer; at.adec.out = a; at.adec.partial = partial;
    at.adec.counters = chunk_counters;
    at.adec.Hq = Hq; at.adec.Hkv = Hkv; at.adec.hd = hd; at.adec.max_chunks = m->max_chunks;
    at.adec.reqs_stable = 1; at.adec.kv_pages = d.kv_pages;
    m->ops.push_back(at);
    Op ap;                                   // causal attention of the step's prompt chunks (none in a pure decode step)
    memset(&ap, 0, sizeof(ap));
    ap.kind = EPARA_K_ATTN_PREFILL; ap.rows_per_req = 1;
    ap.apre.qkv = qkv; ap.apre.q_stride = nq; ap.apre.kv_layer = kv_layer; ap.apre.out = a; ap.apre.kv_pages = d.kv_pages;
    ap.apre.Hq = Hq; ap.apre.Hkv = Hkv; ap.apre.hd = hd;
    m->ops.push_back(ap);
    if (!add_gemm(bl, m, a, Hq * hd, Bcap, w[2], dm, Hq * hd, x, dm, nullptr, EPI_RESID_F32, 1)) return EPARA_E_CUDA;
    add_norm(m, x, dm, h, w[3], nullptr, dm, NORM_RMS, 1e-5f, 1);
    if (!add_gemm(bl, m, h, dm, Bcap, w[4], 2 * F, dm, f, F, nullptr, EPI_SWIGLU, 1)) return EPARA_E_CUDA;
    if (!add_gemm(bl, m, f, F, Bcap, w[5], dm, F, x, dm, nullptr, EPI_RESID_F32, 1)) return EPARA_E_CUDA;
    add_trace(l + 1);
  }
  const void* const* w = t + 1 + 6 * d.n_layers;
  add_norm(m, x, dm, h, w[0], nullptr, dm, NORM_RMS, 1e-5f, 1);
  if (!add_gemm(bl, m, h, dm, Bcap, w[1], d.vocab, dm, logits, ldl, nullptr, 0, 1)) return EPARA_E_CUDA;
  Op o;
  memset(&o, 0, sizeof(o));
  o.kind = EPARA_K_OUTPUT; o.rows_per_req = 1;
  o.outp.logits = logits; o.outp.N = d.vocab; o.outp.ld = ldl;
  m->ops.push_back(o);
  m->n_out = d.vocab;
  // every op up to the last layer works on token rows; the final norm picks each request's last token row
  // and the LM head and the output run per request
  const size_t n_ops = m->ops.size();
  for (size_t i = 0; i + 3 < n_ops; ++i) m->ops[i].per_token = 1;
  m->ops[n_ops - 3].last_rows = 1;
  return EPARA_OK;
}

// Split-k scratch shared by the model's GEMMs (they run one after the other): fp32 partials and
// per-tile arrival counters (zero between launches).
int finish_model(Builder& bl, Model* m) {
  if (m->splitk_bytes == 0) return EPARA_OK;
  float* partial = (float*)bl.get(m->splitk_bytes);
  int* counters = (int*)bl.get(m->splitk_tiles * sizeof(int));
  if (bl.fail) return EPARA_E_RESOURCE;
  if (bl.c) {
    if (cudaMemset(counters, 0, m->splitk_tiles * sizeof(int)) != cudaSuccess) return EPARA_E_CUDA;
    for (Op& op : m->ops)
      if (op.kind == EPARA_K_GEMM && op.gemm.ksplit > 1 && op.gemm.stream == 0) { op.gemm.partial = partial; op.gemm.counters = counters; }
  }
  return EPARA_OK;
}

int effective_max_batch(const epara_config& cfg, const epara_model_desc& d) {
  const int ls = cfg.cap_ls > 0 ? cfg.cap_ls : 4, fs = cfg.cap_fs > 0 ? cfg.cap_fs : 256;
  return d.max_batch > 0 ? d.max_batch : ls + fs;
}

void admit_impl(int n, const uint64_t* tickets, const long long* deadline, const int* streams, long long now, int cap,
                int mf_max, std::vector<int>& admitted, std::vector<int>& dropped) {
  std::vector<int> live;
  for (int i = 0; i < n; ++i) {
    if (deadline[i] != 0 && deadline[i] < now) dropped.push_back(i); else live.push_back(i);
  }
  if (mf_max <= 0) {
    for (int i = 0; i < (int)live.size() && i < cap; ++i) admitted.push_back(live[i]);
    return;
  }
  const int n_streams = cap / mf_max;   // Eq. 5
  std::vector<int> order;
  for (int i : live)
    if (std::find(order.begin(), order.end(), streams[i]) == order.end()) order.push_back(streams[i]);
  if ((int)order.size() > n_streams) order.resize(n_streams);
  if (order.empty()) return;
  int f = mf_max;
  for (int s : order) {
    int cnt = 0;
    for (int i : live) cnt += streams[i] == s;
    f = std::min(f, cnt);
  }
  for (int s : order) {
    int cnt = 0;
    for (int i : live)
      if (streams[i] == s && cnt < f) { admitted.push_back(i); ++cnt; }
  }
  (void)tickets;
}

// Gives every request of the step recorded in `slot` its final answer (the step has finished on the
// device, or never ran) and forgets the step, so that the slot can take another one.
void finalize_slot(epara_ctx* c, Slot& slot) {
  const int code = *slot.status_host;
  for (uint64_t tk : slot.tickets) {
    auto it = c->tickets.find(tk);
    if (it == c->tickets.end() || it->second.state != T_INFLIGHT || it->second.step != slot.step_id) continue;
    Ticket& t = it->second;
    t.state = T_DONE;
    t.device_error = code;
    t.result = code != 0 ? EPARA_E_DEVICE : slot.launch_status;
  }
  slot.tickets.clear();
  slot.busy = false;
}

// A step that fails on the host after admission: its requests answer `result`, nothing stays in flight.
void fail_tickets(epara_ctx* c, const std::vector<uint64_t>& tks, int result) {
  for (uint64_t tk : tks) {
    auto it = c->tickets.find(tk);
    if (it == c->tickets.end()) continue;
    it->second.state = T_DONE;
    it->second.result = result;
    it->second.device_error = 0;
  }
}

}  // namespace

// =============================================================================== C ABI
extern "C" {

const char* epara_strerror(int s) {
  switch (s) {
    case EPARA_OK: return "ok";
    case EPARA_PENDING: return "pending";
    case EPARA_E_INVALID: return "invalid argument";
    case EPARA_E_UNSUPPORTED: return "unsupported (needs more than one GPU, or an unsupported shape)";
    case EPARA_E_TIMEOUT: return "timeout";
    case EPARA_E_RESOURCE: return "resource insufficiency";
    case EPARA_E_DEVICE: return "device-side error";
    case EPARA_E_CUDA: return "CUDA runtime error";
    default: return "unknown status";
  }
}

int epara_dp_group_count(double required_fps, double group_fps) {
  if (!(group_fps > 0) || !(required_fps >= 0)) return EPARA_E_INVALID;
  return (int)std::ceil(required_fps / group_fps);
}

int epara_inter_request_count(int bs, int mf_max) {
  if (bs < 0 || mf_max <= 0) return EPARA_E_INVALID;
  return bs / mf_max;
}

int epara_admit_queue(int n, const uint64_t* tickets, const long long* deadline_ns, const int* streams,
                      long long now_ns, int cap, int mf_max, uint64_t* out_admitted, int* n_admitted,
                      uint64_t* out_dropped, int* n_dropped) {
  if (n < 0 || (n > 0 && (!tickets || !deadline_ns || !streams)) || !n_admitted || !n_dropped || cap < 0)
    return EPARA_E_INVALID;
  std::vector<int> a, d;
  admit_impl(n, tickets, deadline_ns, streams, now_ns, cap, mf_max, a, d);
  for (size_t i = 0; i < a.size(); ++i) out_admitted[i] = tickets[a[i]];
  for (size_t i = 0; i < d.size(); ++i) out_dropped[i] = tickets[d[i]];
  *n_admitted = (int)a.size();
  *n_dropped = (int)d.size();
  return EPARA_OK;
}

size_t epara_model_workspace_bytes(const epara_config* cfg, const epara_model_desc* d) {
  if (!cfg || validate_desc(d) != EPARA_OK) return 0;
  Model m;
  m.d = *d;
  m.tensors.assign(d->tensors, d->tensors + d->n_tensors);
  if (d->kind == EPARA_MODEL_MLP) m.dims.assign(d->mlp_dims, d->mlp_dims + d->n_layers + 1);
  m.max_batch = effective_max_batch(*cfg, *d);
  Builder bl{nullptr, 0, false, device_sm_count(cfg->device), cfg->gemm_impl};
  build_model(bl, &m, *cfg);
  finish_model(bl, &m);
  return bl.need + 256;
}

int epara_init(const epara_config* cfg, epara_ctx** out) {
  if (!cfg || !out) return EPARA_E_INVALID;
  if (!cfg->workspace || (reinterpret_cast<uintptr_t>(cfg->workspace) & 255)) return EPARA_E_INVALID;
  const size_t fixed = N_SLOTS * (BLOB_BYTES + 256);
  if (cfg->workspace_bytes < fixed) return EPARA_E_RESOURCE;
  if (cudaSetDevice(cfg->device) != cudaSuccess) return EPARA_E_CUDA;
  epara_ctx* c = new (std::nothrow) epara_ctx();
  if (!c) return EPARA_E_RESOURCE;
  c->cfg = *cfg;
  if (c->cfg.cap_ls <= 0) c->cfg.cap_ls = 4;
  if (c->cfg.cap_fs <= 0) c->cfg.cap_fs = 256;
  if (c->cfg.max_queue <= 0) c->cfg.max_queue = 4096;
  c->ws = (unsigned char*)cfg->workspace;
  c->ws_bytes = cfg->workspace_bytes;
  c->ws_used = 0;
  c->next_ticket = 1;
  c->next_step = 1;
  c->last_step_slot = 0;
  c->max_profile_launches = MAX_PROFILE_LAUNCHES;
  int sm = 0;
  if (cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess) { delete c; return EPARA_E_CUDA; }
  c->sm_count = sm;
  for (int i = 0; i < N_SLOTS; ++i) {
    Slot& s = c->slots[i];
    s.dev = (unsigned char*)carve(c, BLOB_BYTES);
    s.step_id = 0;
    s.busy = false;
    s.profiled = false;
    s.launch_status = EPARA_OK;
    if (cudaMallocHost((void**)&s.host, BLOB_BYTES) != cudaSuccess ||
        cudaMallocHost((void**)&s.status_host, 64) != cudaSuccess ||
        cudaEventCreateWithFlags(&s.done, cudaEventDisableTiming) != cudaSuccess) {
      return EPARA_E_CUDA;
    }
    *s.status_host = 0;
  }
  *out = c;
  return EPARA_OK;
}

int epara_destroy(epara_ctx* c) {
  if (!c) return EPARA_E_INVALID;
  cudaSetDevice(c->cfg.device);
  for (int i = 0; i < N_SLOTS; ++i) {
    Slot& s = c->slots[i];
    if (s.busy) cudaEventSynchronize(s.done);
    for (cudaEvent_t e : s.prof) cudaEventDestroy(e);
    cudaEventDestroy(s.done);
    cudaFreeHost(s.host);
    cudaFreeHost(s.status_host);
  }
  for (Model* m : c->models) delete m;
  delete c;
  return EPARA_OK;
}

int epara_register_model(epara_ctx* c, const epara_model_desc* d, int* model_id) {
  if (!c || !model_id) return EPARA_E_INVALID;
  int v = validate_desc(d);
  if (v != EPARA_OK) return v;
  if (cudaSetDevice(c->cfg.device) != cudaSuccess) return EPARA_E_CUDA;
  Model* m = new (std::nothrow) Model();
  if (!m) return EPARA_E_RESOURCE;
  m->d = *d;
  m->tensors.assign(d->tensors, d->tensors + d->n_tensors);
  if (d->kind == EPARA_MODEL_MLP) m->dims.assign(d->mlp_dims, d->mlp_dims + d->n_layers + 1);
  m->d.tensors = nullptr;
  m->d.mlp_dims = nullptr;
  m->max_batch = effective_max_batch(c->cfg, *d);
  m->max_chunks = 0;
  m->kv_bytes_per_token = 0;
  const size_t mark = c->ws_used;
  Builder bl{c, 0, false, c->sm_count, c->cfg.gemm_impl};
  int r = build_model(bl, m, c->cfg);
  if (r == EPARA_OK) r = finish_model(bl, m);
  if (r != EPARA_OK) {
    c->ws_used = mark;
    delete m;
    return r;
  }
  c->models.push_back(m);
  *model_id = (int)c->models.size() - 1;
  return EPARA_OK;
}

int epara_submit(epara_ctx* c, int model_id, int category, const epara_inputs* in, uint64_t* ticket) {
  if (!c || !in || !ticket) return EPARA_E_INVALID;
  if (model_id < 0 || model_id >= (int)c->models.size()) return EPARA_E_INVALID;
  if (category == EPARA_CAT_LS_GT1 || category == EPARA_CAT_FS_GT1) return EPARA_E_UNSUPPORTED;
  if (category != EPARA_CAT_LS_LT1 && category != EPARA_CAT_FS_LT1) return EPARA_E_INVALID;
  Model* m = c->models[model_id];
  if (!in->out_logits && !in->out_argmax) return EPARA_E_INVALID;
  if (reinterpret_cast<uintptr_t>(in->out_logits) & 1) return EPARA_E_INVALID;
  const int n_tok = (m->d.kind == EPARA_MODEL_DECODER && in->n_tokens > 1) ? in->n_tokens : 1;
  if (m->d.kind == EPARA_MODEL_DECODER) {
    if (in->n_tokens < 0 || (in->n_tokens > 1 && !in->tokens)) return EPARA_E_INVALID;
    const long long last_pos = (long long)in->kv_len + n_tok - 1;         // position of the request's last token
    if (!in->block_table || in->kv_len < 0 || last_pos > m->d.max_kv_len) return EPARA_E_INVALID;
    if (in->n_blocks < last_pos / EPARA_KV_PAGE + 1) return EPARA_E_INVALID;
    if (n_tok > m->max_batch) return EPARA_E_RESOURCE;                      // more token rows than the model was placed for
    if (n_tok > 1) {
      if (m->d.head_dim != 64 && m->d.head_dim != 128) return EPARA_E_UNSUPPORTED;
      for (int i = 0; i < n_tok; ++i)
        if (in->tokens[i] < 0 || in->tokens[i] >= m->d.vocab) return EPARA_E_INVALID;
    } else if (in->n_tokens == 1 && in->tokens) {
      if (in->tokens[0] < 0 || in->tokens[0] >= m->d.vocab) return EPARA_E_INVALID;
    } else if (in->token < 0 || in->token >= m->d.vocab) {
      return EPARA_E_INVALID;
    }
  } else {
    if (!in->input || (reinterpret_cast<uintptr_t>(in->input) & 15)) return EPARA_E_INVALID;
  }
  if ((int)m->q[category].size() >= c->cfg.max_queue) return EPARA_E_RESOURCE;
  Request r;
  r.ticket = c->next_ticket++;
  r.in = *in;
  if (m->d.kind == EPARA_MODEL_DECODER) {
    if (n_tok > 1) r.toks.assign(in->tokens, in->tokens + n_tok);
    else if (in->n_tokens == 1 && in->tokens) r.in.token = in->tokens[0];
    r.in.tokens = nullptr;                 // the caller's array is not kept
  }
  m->q[category].push_back(std::move(r));
  Ticket t;
  t.state = T_QUEUED; t.model = model_id; t.step = 0; t.out_logits = in->out_logits; t.out_argmax = in->out_argmax;
  t.result = EPARA_OK; t.device_error = 0;
  c->tickets[r.ticket] = t;
  *ticket = r.ticket;
  return EPARA_OK;
}

int epara_submit_many(epara_ctx* c, int model_id, int category, const epara_inputs* in, int n, uint64_t* tickets,
                      int* n_accepted) {
  if (n_accepted) *n_accepted = 0;
  if (!c || n < 0 || (n > 0 && (!in || !tickets))) return EPARA_E_INVALID;
  for (int i = 0; i < n; ++i) {
    const int r = epara_submit(c, model_id, category, in + i, tickets + i);
    if (r != EPARA_OK) return r;
    if (n_accepted) *n_accepted = i + 1;
  }
  return EPARA_OK;
}

int epara_step(epara_ctx* c, void* cuda_stream, long long now_ns, epara_step_info* info) {
  if (!c) return EPARA_E_INVALID;
  if (cudaSetDevice(c->cfg.device) != cudaSuccess) return EPARA_E_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (now_ns < 0)
    now_ns = std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now().time_since_epoch()).count();
  epara_step_info inf;
  memset(&inf, 0, sizeof(inf));
  const uint64_t step_id = c->next_step++;
  inf.step_id = step_id;

  // ---- admission (A0) ----
  // B requests; `rows` activation rows (one per token for a decoder, B otherwise); n_dec single-token and
  // n_pre prompt-chunk requests of a decoder, with their descriptor arrays in the blob
  struct Active {
    Model* m; int B; int rows; size_t req_off; size_t areq_off; size_t row_off; size_t preq_off; size_t last_off; size_t cursor;
    int n_dec, n_pre, max_chunks_dec, pre_blocks;
    std::vector<Request> reqs;
  };
  std::vector<Active> act;
  for (size_t mi = 0; mi < c->models.size(); ++mi) {
    Model* m = c->models[mi];
    Active a;
    a.m = m; a.B = 0; a.rows = 0; a.cursor = 0; a.req_off = 0; a.areq_off = 0; a.row_off = 0; a.preq_off = 0; a.last_off = 0;
    a.n_dec = a.n_pre = a.max_chunks_dec = a.pre_blocks = 0;
    for (int cat = 0; cat < 2; ++cat) {
      std::deque<Request>& q = m->q[cat];
      if (q.empty()) continue;
      const int n = (int)q.size();
      std::vector<uint64_t> tk(n);
      std::vector<long long> dl(n);
      std::vector<int> sid(n);
      for (int i = 0; i < n; ++i) { tk[i] = q[i].ticket; dl[i] = q[i].in.deadline_ns; sid[i] = q[i].in.stream; }
      int cap = (cat == EPARA_CAT_LS_LT1) ? c->cfg.cap_ls : c->cfg.cap_fs;
      cap = std::min(cap, m->max_batch - a.B);
      std::vector<int> adm, drp;
      admit_impl(n, tk.data(), dl.data(), sid.data(), now_ns, cap, (cat == EPARA_CAT_FS_LT1) ? c->cfg.mf_max : 0, adm, drp);
      // a request takes one activation row per token: admitted requests beyond the model's rows wait for a later step
      {
        size_t keep = 0;
        for (; keep < adm.size(); ++keep) {
          const int nt = q[adm[keep]].n_tok();
          if (a.rows + nt > m->max_batch) break;
          a.rows += nt;
        }
        adm.resize(keep);
      }
      std::vector<char> gone(n, 0);
      for (int i : adm) { a.reqs.push_back(q[i]); gone[i] = 1; c->tickets[q[i].ticket].state = T_INFLIGHT; c->tickets[q[i].ticket].step = step_id; }
      for (int i : drp) { gone[i] = 1; Ticket& t = c->tickets[q[i].ticket]; t.state = T_DONE; t.result = EPARA_E_TIMEOUT; }
      std::deque<Request> rest;
      for (int i = 0; i < n; ++i) if (!gone[i]) rest.push_back(q[i]);
      q.swap(rest);
      inf.admitted[cat] += (int)adm.size();
      inf.dropped[cat] += (int)drp.size();
      a.B += (int)adm.size();
    }
    if (a.B > 0) act.push_back(std::move(a));
  }
  if (act.empty()) {
    if (info) *info = inf;
    return EPARA_OK;
  }

  // ---- blob slot ----
  std::vector<uint64_t> admitted_tickets;
  for (Active& a : act)
    for (Request& r : a.reqs) admitted_tickets.push_back(r.ticket);
  Slot& slot = c->slots[step_id % N_SLOTS];
  if (slot.busy) {
    // the step that used this slot N_SLOTS steps ago: wait for it and give its requests their answers
    if (cudaEventSynchronize(slot.done) != cudaSuccess) {
      fail_tickets(c, admitted_tickets, EPARA_E_CUDA);
      if (info) *info = inf;
      return EPARA_E_CUDA;
    }
  }
  if (!slot.tickets.empty()) finalize_slot(c, slot);
  slot.busy = false;
  memset(slot.host, 0, BLOB_HEADER);         // the step's status word, cleared on the device by the upload
  int* const dev_status = reinterpret_cast<int*>(slot.dev);
  size_t off = BLOB_HEADER;
  auto put = [&](const void* src, size_t bytes, size_t align) -> size_t {
    off = align_up(off, align);
    if (off + bytes > BLOB_BYTES) return (size_t)-1;
    memcpy(slot.host + off, src, bytes);
    const size_t at = off;
    off += bytes;
    return at;
  };
  bool overflow = false;
  for (Active& a : act) {
    const bool dec = a.m->d.kind == EPARA_MODEL_DECODER;
    std::vector<ReqDesc> rd(a.B);
    std::vector<AttnReq> ar;
    std::vector<PrefillReq> pr;
    std::vector<RowDesc> rows;
    std::vector<int> last(a.B);
    int row = 0;
    for (int b = 0; b < a.B; ++b) {
      const Request& rq = a.reqs[b];
      const epara_inputs& in = rq.in;
      const int nt = dec ? rq.n_tok() : 1;
      memset(&rd[b], 0, sizeof(ReqDesc));
      rd[b].input = in.input; rd[b].table = in.block_table; rd[b].out_logits = in.out_logits;
      rd[b].out_argmax = in.out_argmax; rd[b].token = in.token; rd[b].kv_len = in.kv_len;
      rd[b].n_blocks = in.n_blocks; rd[b].row_start = row; rd[b].n_tok = nt;
      if (dec) {
        for (int t = 0; t < nt; ++t) {
          RowDesc r;
          r.req = b; r.pos = in.kv_len + t; r.token = nt > 1 ? rq.toks[t] : in.token; r.pad = 0;
          rows.push_back(r);
        }
        if (nt == 1) {
          AttnReq q1;
          q1.table = in.block_table; q1.len = in.kv_len + 1; q1.row = row;
          ar.push_back(q1);
          a.max_chunks_dec = std::max(a.max_chunks_dec, (in.kv_len + 1 + ATTN_CHUNK - 1) / ATTN_CHUNK);
        } else {
          PrefillReq p1;
          p1.table = in.block_table; p1.row_start = row; p1.n_tok = nt; p1.kv_len = in.kv_len; p1.blk_start = a.pre_blocks;
          a.pre_blocks += attn_prefill_blocks(nt, a.m->d.n_heads);
          pr.push_back(p1);
          inf.prefill_tokens += nt;
        }
        // cached bytes the step must read at least once: the request's whole sequence, once per layer
        inf.kv_bytes += a.m->kv_bytes_per_token * (in.kv_len + (nt > 1 ? nt : 0));
      }
      last[b] = row + nt - 1;
      row += nt;
    }
    a.rows = dec ? row : a.B;
    a.n_dec = (int)ar.size(); a.n_pre = (int)pr.size();
    a.req_off = put(rd.data(), rd.size() * sizeof(ReqDesc), 16);
    if (dec) {
      a.row_off = put(rows.data(), rows.size() * sizeof(RowDesc), 16);
      a.last_off = put(last.data(), last.size() * sizeof(int), 16);
      if (!ar.empty()) a.areq_off = put(ar.data(), ar.size() * sizeof(AttnReq), 16);
      if (!pr.empty()) a.preq_off = put(pr.data(), pr.size() * sizeof(PrefillReq), 16);
    }
    if (a.req_off == (size_t)-1 || a.areq_off == (size_t)-1 || a.row_off == (size_t)-1 || a.preq_off == (size_t)-1 ||
        a.last_off == (size_t)-1)
      overflow = true;
  }

  // ---- plan (A1): sweep the kernel kinds until every model's op list is exhausted ----
  static const int sweep[] = {EPARA_K_GATHER, EPARA_K_TRACE, EPARA_K_ASSEMBLE, EPARA_K_NORM, EPARA_K_GEMM, EPARA_K_ROPE,
                              EPARA_K_ATTN_DEC, EPARA_K_ATTN_PREFILL, EPARA_K_ATTN_ENC, EPARA_K_OUTPUT};
  std::vector<Launch> launches;
  const bool simt = c->cfg.gemm_impl == EPARA_GEMM_SIMT;
  bool more = true;
  while (more && !overflow) {
    more = false;
    for (int kind : sweep) {
      std::vector<Active*> who;
      for (Active& a : act)
        if (a.cursor < a.m->ops.size() && a.m->ops[a.cursor].kind == kind) who.push_back(&a);
      if (who.empty()) continue;
      more = true;
      if (kind == EPARA_K_TRACE) {               // debug copies of the residual stream: one plain copy per model
        for (Active* a : who) {
          const Op& op = a->m->ops[a->cursor];
          Launch LL;
          memset(&LL, 0, sizeof(LL));
          LL.kind = kind; LL.n_groups = 1;
          LL.src = op.trace_src; LL.dst = op.trace_dst; LL.bytes = (size_t)a->rows * op.trace_row_bytes;
          launches.push_back(LL);
          a->cursor++;
        }
        continue;
      }
      // GEMM groups go out in up to three launches: tensor-core tiles (pass 0), the weight-streaming
      // kernel for groups that never exceed 16 rows (pass 1) and 256-row tiles on CTA pairs for the dense
      // bf16-output groups (pass 2); encoder attention in two: the tcgen05 kernel (pass 0) and the
      // mma.sync kernel for shapes it does not take (pass 1)
      // (passes 3 to 6: the swapped-operand kernel with 1, 2, 4 and 8 k ranges per tile)
      // (pass 7: encoder MLP blocks in the fused kernel)
      const int n_pass = kind == EPARA_K_GEMM ? 8 : (kind == EPARA_K_ATTN_ENC ? 2 : 1);
      for (int pass = 0; pass < n_pass; ++pass) {
      Launch L;
      memset(&L, 0, sizeof(L));
      L.kind = kind;
      L.n_groups = (int)who.size();
      L.p2 = pass;
      int n_put = 0;
      off = align_up(off, 64);
      L.off = off;
      if (kind == EPARA_K_ATTN_DEC) {
        // decode attention is templated on (hd, G): one launch per distinct pair
        std::vector<Active*> rest = who;
        while (!rest.empty()) {
          const Op& o0 = rest[0]->m->ops[rest[0]->cursor];
          const int hd = o0.adec.hd, G = o0.adec.Hq / o0.adec.Hkv;
          std::vector<Active*> same, other;
          for (Active* a : rest) {
            const Op& o = a->m->ops[a->cursor];
            ((o.adec.hd == hd && o.adec.Hq / o.adec.Hkv == G) ? same : other).push_back(a);
          }
          Launch LL;
          memset(&LL, 0, sizeof(LL));
          LL.kind = kind; LL.n_groups = (int)same.size();
          off = align_up(off, 64);
          LL.off = off;
          int total_B = 0, max_hkv = 0, max_hq = 0, max_chunks = 0, n_put = 0;
          for (Active* a : same) {
            if (a->n_dec == 0) continue;               // only prompt chunks from this model in this step
            AttnDecGroup g = a->m->ops[a->cursor].adec;
            g.B = a->n_dec; g.reqs = (const AttnReq*)(slot.dev + a->areq_off); g.req_start = total_B;
            g.status = dev_status;
            total_B += a->n_dec;
            max_hkv = std::max(max_hkv, g.Hkv); max_hq = std::max(max_hq, g.Hq);
            max_chunks = std::max(max_chunks, a->max_chunks_dec);
            ++n_put;
            if (put(&g, sizeof(g), 8) == (size_t)-1) overflow = true;
          }
          LL.n_groups = n_put;
          LL.p0 = total_B; LL.p1 = max_hkv | (max_hq << 16); LL.p2 = max_chunks; LL.p3 = (hd << 8) | G;
          if (n_put > 0) launches.push_back(LL);
          rest.swap(other);
        }
        for (Active* a : who) a->cursor++;
        continue;
      }
      if (kind == EPARA_K_ATTN_PREFILL) {
        for (int hd : {64, 128}) {
          Launch LL;
          memset(&LL, 0, sizeof(LL));
          LL.kind = kind;
          off = align_up(off, 64);
          LL.off = off;
          int blocks = 0, n_put = 0;
          for (Active* a : who) {
            AttnPrefillGroup g = a->m->ops[a->cursor].apre;
            if (g.hd != hd || a->n_pre == 0) continue;
            g.reqs = (const PrefillReq*)(slot.dev + a->preq_off); g.n_reqs = a->n_pre; g.status = dev_status;
            g.blk_start = blocks; g.n_blocks = a->pre_blocks;
            blocks += a->pre_blocks;
            ++n_put;
            if (put(&g, sizeof(g), 8) == (size_t)-1) overflow = true;
          }
          LL.n_groups = n_put; LL.p0 = blocks; LL.p1 = hd;
          if (n_put > 0) launches.push_back(LL);
        }
        for (Active* a : who) a->cursor++;
        continue;
      }
      int total = 0, mx = 0;
      for (Active* a : who) {
        const Op& op = a->m->ops[a->cursor];
        const int rows = op.per_token ? a->rows : a->B * op.rows_per_req;
        switch (kind) {
          case EPARA_K_GATHER: {
            GatherGroup g = op.gather;
            g.reqs = (const ReqDesc*)(slot.dev + a->req_off); g.B = a->B;
            g.rows = (const RowDesc*)(slot.dev + a->row_off);
            g.blocks = g.kind == GATHER_PATCH ? (rows + GATHER_PATCH_ROWS - 1) / GATHER_PATCH_ROWS : rows;
            mx = std::max(mx, g.blocks);
            if (put(&g, sizeof(g), 8) == (size_t)-1) overflow = true;
            break;
          }
          case EPARA_K_ASSEMBLE: {
            AssembleGroup g = op.asmb;
            g.B = a->B;
            mx = std::max(mx, rows);
            if (put(&g, sizeof(g), 8) == (size_t)-1) overflow = true;
            break;
          }
          case EPARA_K_NORM: {
            NormGroup g = op.norm;
            g.M = rows;
            if (op.last_rows) g.row_index = (const int*)(slot.dev + a->last_off);
            mx = std::max(mx, norm_blocks(rows, g.d));
            if (put(&g, sizeof(g), 8) == (size_t)-1) overflow = true;
            break;
          }
          case EPARA_K_GEMM: {
            GemmGroup g = op.gemm;
            int gpass = g.stream;
            if (g.stream == 3) gpass = 3 + (g.ksplit >= 8 ? 3 : g.ksplit >= 4 ? 2 : g.ksplit >= 2 ? 1 : 0);
            if (g.stream == 4) gpass = 7;
            if (gpass != pass) break;                          // another pass takes it
            if (g.stream == 4) {
              MlpGroup mg = op.mlp;
              mg.M = rows;
              mg.tiles_m = (rows + 2 * TC_BM - 1) / (2 * TC_BM);
              mg.tile_start = total;
              total += mg.tiles_m;
              ++n_put;
              inf.gemm_groups++;
              inf.gemm_flops += 2.0 * 2.0 * rows * mg.d * mg.F;
              inf.weight_bytes += op.weight_bytes;
              if (put(&mg, sizeof(mg), 64) == (size_t)-1) overflow = true;
              break;
            }
            g.M = rows;
            if (g.stream == 3) {
              g.tiles_m = 1; g.tiles_n = gemm_swap_tiles(g.N);
              g.tile_start = total;
              total += g.tiles_n;
            } else if (g.stream == 2) {
              g.tiles_m = (rows + 2 * TC_BM - 1) / (2 * TC_BM); g.tiles_n = (g.N + g.bn - 1) / g.bn;
              g.tile_start = total;
              total += g.tiles_m * g.tiles_n;
            } else if (g.stream) {
              g.tiles_m = 1; g.tiles_n = gemm_stream_tiles(g.N);
              g.tile_start = total;
              total += g.tiles_n;
              mx = std::max(mx, rows);
            } else {
              const int tm = simt ? SIMT_TILE : TC_BM, tn = simt ? SIMT_TILE : g.bn;
              g.tiles_m = (rows + tm - 1) / tm; g.tiles_n = (g.N + tn - 1) / tn;
              g.tile_start = total;
              total += g.tiles_m * g.tiles_n * (simt ? 1 : g.ksplit);
              L.p3 = std::max(L.p3, g.bn);
            }
            ++n_put;
            inf.gemm_groups++;
            inf.gemm_flops += 2.0 * rows * g.N * g.K;
            inf.weight_bytes += op.weight_bytes;
            if (g.stream == 1) {
              inf.stream_gemm_flops += 2.0 * rows * g.N * g.K;
              inf.stream_weight_bytes += op.weight_bytes;
            }
            if (put(&g, sizeof(g), 64) == (size_t)-1) overflow = true;
            break;
          }
          case EPARA_K_ROPE: {
            RopeGroup g = op.rope;
            g.reqs = (const ReqDesc*)(slot.dev + a->req_off); g.B = rows;
            g.rows = (const RowDesc*)(slot.dev + a->row_off);
            g.status = dev_status;
            mx = std::max(mx, rows);
            if (put(&g, sizeof(g), 8) == (size_t)-1) overflow = true;
            break;
          }
          case EPARA_K_ATTN_ENC: {
            AttnEncGroup g = op.aenc;
            if ((g.tc != 0) != (pass == 0)) break;             // the other pass takes it
            g.B = a->B; g.q_blocks = g.tc ? 1 : attn_encoder_q_blocks(g.T); g.blk_start = total;
            total += a->B * g.H * g.q_blocks;
            mx = std::max(mx, g.T);
            ++n_put;
            if (put(&g, sizeof(g), 64) == (size_t)-1) overflow = true;
            break;
          }
          case EPARA_K_OUTPUT: {
            OutputGroup g = op.outp;
            g.reqs = (const ReqDesc*)(slot.dev + a->req_off); g.B = a->B;
            mx = std::max(mx, a->B);
            if (put(&g, sizeof(g), 8) == (size_t)-1) overflow = true;
            break;
          }
        }
        if (pass == n_pass - 1) a->cursor++;
      }
      L.p0 = total; L.p1 = mx;
      if (kind == EPARA_K_GEMM || kind == EPARA_K_ATTN_ENC) {
        L.n_groups = n_put;
        if (n_put == 0) continue;
      }
      launches.push_back(L);
      }
    }
  }
  // Every exit from here on that launches nothing gives the admitted requests a definite answer.
  auto fail = [&](int result) {
    fail_tickets(c, admitted_tickets, result);
    if (info) *info = inf;
    return result;
  };
  if (overflow) return fail(EPARA_E_RESOURCE);     // the step's descriptors do not fit the blob
  const bool prof = c->cfg.profile != 0;
  if (prof) {
    if ((int)launches.size() > c->max_profile_launches) return fail(EPARA_E_RESOURCE);
    while (slot.prof.size() < 2 * launches.size()) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return fail(EPARA_E_CUDA);
      slot.prof.push_back(e);
    }
    slot.prof_kind.clear();
  }

  // ---- upload + launch ----
  if (cudaMemcpyAsync(slot.dev, slot.host, off, cudaMemcpyHostToDevice, st) != cudaSuccess) return fail(EPARA_E_CUDA);
  slot.profiled = prof;
  cudaError_t err = cudaSuccess;
  int li = 0, n_kernels = 0;
  for (const Launch& L : launches) {
    n_kernels += 1 + ((L.kind == EPARA_K_ATTN_DEC && L.p2 > 1 &&
                       !attn_decode_fused(L.p0, L.p1 & 0xffff, L.p2, c->sm_count)) ? 1 : 0);
    const unsigned char* gp = slot.dev + L.off;
    if (prof) {
      cudaEventRecord(slot.prof[2 * li], st);
      slot.prof_kind.push_back(L.kind == EPARA_K_GEMM && L.p2 == 1 ? (int)EPARA_K_GEMM_STREAM : L.kind);
    }
    switch (L.kind) {
      case EPARA_K_GATHER: launch_gather((const GatherGroup*)gp, L.n_groups, L.p1, st); break;
      case EPARA_K_ASSEMBLE: launch_assemble((const AssembleGroup*)gp, L.n_groups, L.p1, st); break;
      case EPARA_K_NORM: launch_norm((const NormGroup*)gp, L.n_groups, L.p1, st); break;
      case EPARA_K_GEMM:
        if (L.p2 == 7) err = launch_gemm_mlp_pair((const MlpGroup*)gp, L.n_groups, L.p0, dev_status, c->sm_count, st);
        else if (L.p2 >= 3) err = launch_gemm_swap((const GemmGroup*)gp, L.n_groups, L.p0, 1 << (L.p2 - 3), dev_status, c->sm_count, st);
        else if (L.p2 == 1) err = launch_gemm_stream((const GemmGroup*)gp, L.n_groups, L.p0, L.p1, st);
        else if (L.p2 == 2) err = launch_gemm_tc_pair((const GemmGroup*)gp, L.n_groups, L.p0, dev_status, c->sm_count, st);
        else if (simt) launch_gemm_simt((const GemmGroup*)gp, L.n_groups, L.p0, st);
        else err = launch_gemm_tc((const GemmGroup*)gp, L.n_groups, L.p0, L.p3, dev_status, c->sm_count, st);
        break;
      case EPARA_K_ROPE: launch_rope_append((const RopeGroup*)gp, L.n_groups, L.p1, st); break;
      case EPARA_K_ATTN_DEC:
        err = launch_attn_decode((const AttnDecGroup*)gp, L.n_groups, L.p0, L.p1 & 0xffff, L.p1 >> 16, L.p2, L.p3 >> 8,
                                 L.p3 & 255, attn_decode_fused(L.p0, L.p1 & 0xffff, L.p2, c->sm_count) ? 1 : 0, st);
        break;
      case EPARA_K_ATTN_ENC:
        if (L.p2 == 0) err = launch_attn_encoder_tc((const AttnEncGroup*)gp, L.n_groups, L.p0, dev_status, c->sm_count, st);
        else err = launch_attn_encoder((const AttnEncGroup*)gp, L.n_groups, L.p0, L.p1, st);
        break;
      case EPARA_K_OUTPUT: launch_output((const OutputGroup*)gp, L.n_groups, L.p1, st); break;
      case EPARA_K_TRACE: err = cudaMemcpyAsync(L.dst, L.src, L.bytes, cudaMemcpyDeviceToDevice, st); break;
      case EPARA_K_ATTN_PREFILL:
        err = launch_attn_prefill((const AttnPrefillGroup*)gp, L.n_groups, L.p0, L.p1, st);
        break;
    }
    if (prof) cudaEventRecord(slot.prof[2 * li + 1], st);
    ++li;
    if (err != cudaSuccess) break;
  }
  if (err == cudaSuccess) err = cudaGetLastError();
  // A launch that failed leaves the step incomplete: the kernels already enqueued still run, the event
  // still fires, and the step's requests then answer EPARA_E_CUDA instead of EPARA_OK.
  slot.launch_status = err == cudaSuccess ? EPARA_OK : EPARA_E_CUDA;
  *slot.status_host = 0;
  if (cudaMemcpyAsync(slot.status_host, dev_status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaEventRecord(slot.done, st) != cudaSuccess)
    slot.launch_status = EPARA_E_CUDA;
  slot.busy = true;
  slot.step_id = step_id;
  slot.tickets = admitted_tickets;
  c->last_step_slot = step_id % N_SLOTS;
  inf.launches = n_kernels;
  if (info) *info = inf;
  return slot.launch_status;
}

int epara_collect(epara_ctx* c, uint64_t ticket, epara_output* out) {
  if (!c) return EPARA_E_INVALID;
  auto it = c->tickets.find(ticket);
  if (it == c->tickets.end()) return EPARA_E_INVALID;
  if (it->second.state == T_QUEUED) return EPARA_PENDING;
  if (it->second.state == T_INFLIGHT) {
    Slot& s = c->slots[it->second.step % N_SLOTS];
    if (s.step_id == it->second.step && s.busy) {
      cudaError_t e = cudaEventQuery(s.done);
      if (e == cudaErrorNotReady) return EPARA_PENDING;
      if (e != cudaSuccess) { s.launch_status = EPARA_E_CUDA; *s.status_host = 0; }
      finalize_slot(c, s);            // answers every request of that step, this one included
    }
    if (it->second.state != T_DONE) {   // (cannot happen: an in-flight ticket's step is always in its slot)
      it->second.state = T_DONE;
      it->second.result = EPARA_E_CUDA;
    }
  }
  const Ticket t = it->second;
  if (out) {
    out->status = t.result;
    out->step_id = t.step;
    out->logits = t.out_logits;
    out->argmax = t.out_argmax;
    out->n_out = c->models[t.model]->n_out;
    out->device_error = t.device_error;
  }
  c->tickets.erase(it);
  return t.result;
}

int epara_set_max_profile_launches(epara_ctx* c, int n) {
  if (!c || n < 0) return EPARA_E_INVALID;
  c->max_profile_launches = n;
  return EPARA_OK;
}

int epara_set_profile(epara_ctx* c, int on) {
  if (!c) return EPARA_E_INVALID;
  c->cfg.profile = on ? 1 : 0;
  return EPARA_OK;
}

int epara_step_profile(epara_ctx* c, float* ms_per_kind, int* launches_per_kind) {
  if (!c || !ms_per_kind || !launches_per_kind) return EPARA_E_INVALID;
  Slot& s = c->slots[c->last_step_slot];
  if (s.step_id == 0 || !s.profiled) return EPARA_E_UNSUPPORTED;
  if (cudaEventSynchronize(s.done) != cudaSuccess) return EPARA_E_CUDA;
  for (int k = 0; k < EPARA_K_COUNT; ++k) { ms_per_kind[k] = 0.f; launches_per_kind[k] = 0; }
  for (size_t i = 0; i < s.prof_kind.size(); ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, s.prof[2 * i], s.prof[2 * i + 1]) != cudaSuccess) return EPARA_E_CUDA;
    ms_per_kind[s.prof_kind[i]] += ms;
    launches_per_kind[s.prof_kind[i]]++;
  }
  return EPARA_OK;
}

// ---------------------------------------------------------------- single-kernel entry points
size_t epara_gemm_scratch_bytes(int n) { return (size_t)(n > 0 ? n : 0) * sizeof(GemmGroup) + 256; }

size_t epara_gemm_scratch_bytes_for(int device, const epara_gemm_problem* p, int n) {
  const int sm_count = device_sm_count(device);
  size_t bytes = epara_gemm_scratch_bytes(n);
  for (int i = 0; i < n && p; ++i) {
    int bn = 128, ks = 1;
    gemm_tc_config(p[i].M, p[i].N, p[i].K, p[i].epilogue, sm_count, &bn, &ks);
    if (ks > 1) {
      const size_t tiles_m = (size_t)(p[i].M + TC_BM - 1) / TC_BM, tiles_n = (size_t)(p[i].N + bn - 1) / bn;
      bytes = align_up(bytes, 256) + (size_t)ks * tiles_m * TC_BM * tiles_n * bn * 4;
      bytes = align_up(bytes, 256) + tiles_m * tiles_n * sizeof(int);
    }
  }
  return bytes;
}

int epara_grouped_gemm(int device, void* cuda_stream, int impl, const epara_gemm_problem* p, int n, void* scratch,
                       size_t scratch_bytes) {
  if (n < 0 || (n > 0 && !p) || !scratch || (reinterpret_cast<uintptr_t>(scratch) & 255)) return EPARA_E_INVALID;
  if (scratch_bytes < (impl == EPARA_GEMM_SIMT ? epara_gemm_scratch_bytes(n) : epara_gemm_scratch_bytes_for(device, p, n)))
    return EPARA_E_RESOURCE;
  if (n == 0) return EPARA_OK;
  if (cudaSetDevice(device) != cudaSuccess) return EPARA_E_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const bool simt = impl == EPARA_GEMM_SIMT;
  const int sm_count = device_sm_count(device);
  std::vector<GemmGroup> gs, gs_stream, gs_pair;   // tensor-core (or CUDA-core) groups; weight-streaming groups (M <= 16); CTA-pair groups
  std::vector<GemmGroup> gs_swap[4];               // swapped-operand groups (17 to 128 rows) by k ranges per tile: 1, 2, 4, 8
  int total_swap[4] = {0, 0, 0, 0};
  int total = 0, total_stream = 0, max_rows_stream = 0, total_pair = 0;
  size_t soff = epara_gemm_scratch_bytes(n);
  for (int i = 0; i < n; ++i) {
    const epara_gemm_problem& q = p[i];
    if (!q.A || !q.W || !q.C || q.M < 0 || q.N <= 0 || q.K <= 0) return EPARA_E_INVALID;
    if ((q.lda % 8) || (q.ldw % 8) || q.lda < q.K || q.ldw < q.K) return EPARA_E_INVALID;
    if ((reinterpret_cast<uintptr_t>(q.A) & 15) || (reinterpret_cast<uintptr_t>(q.W) & 15) ||
        (reinterpret_cast<uintptr_t>(q.C) & 15))
      return EPARA_E_INVALID;
    if ((q.epilogue & EPARA_EPI_SWIGLU) && (q.N % 2 || (q.epilogue & EPARA_EPI_RESID_F32))) return EPARA_E_INVALID;
    if ((q.epilogue & EPARA_EPI_BIAS) && !q.bias) return EPARA_E_INVALID;
    GemmGroup g;
    memset(&g, 0, sizeof(g));
    g.A = (const bf16*)q.A; g.W = (const bf16*)q.W; g.C = q.C; g.bias = (const bf16*)q.bias;
    g.M = q.M; g.N = q.N; g.K = q.K; g.lda = q.lda; g.ldw = q.ldw; g.ldc = q.ldc; g.epi = q.epilogue;
    g.bn = 128; g.ksplit = 1;
    g.c_rows = q.M;
    if (!simt && q.M <= GEMM_STREAM_MAX_ROWS && q.K % 8 == 0) {
      g.stream = 1; g.bn = 16;
      g.tiles_m = 1; g.tiles_n = gemm_stream_tiles(q.N);
      g.tile_start = total_stream;
      if (q.M > 0) total_stream += g.tiles_n;
      max_rows_stream = std::max(max_rows_stream, q.M);
      gs_stream.push_back(g);
      continue;
    }
    if (!simt && q.M <= GEMM_SWAP_MAX_ROWS && q.K % 8 == 0) {
      g.stream = 3;
      g.bn = round_up(q.M, 16);
      g.ksplit = gemm_swap_ksplit(q.N, q.K, sm_count);
      const int si = g.ksplit >= 8 ? 3 : g.ksplit >= 4 ? 2 : g.ksplit >= 2 ? 1 : 0;
      g.tiles_m = 1; g.tiles_n = gemm_swap_tiles(q.N);
      g.tile_start = total_swap[si];
      total_swap[si] += g.tiles_n;
      if (!make_tmap(&g.tmA, q.A, q.M, q.K, q.lda, g.bn)) return EPARA_E_CUDA;
      if (!make_tmap(&g.tmW, q.W, q.N, q.K, q.ldw, TC_BM)) return EPARA_E_CUDA;
      gs_swap[si].push_back(g);
      continue;
    }
    if (!simt) gemm_tc_config(q.M, q.N, q.K, q.epilogue, sm_count, &g.bn, &g.ksplit);
    if (!simt && gemm_tc_pair_eligible(q.M, q.N, q.K, q.epilogue, g.bn, g.ksplit)) {
      g.stream = 2;
      g.tiles_m = (q.M + 2 * TC_BM - 1) / (2 * TC_BM); g.tiles_n = (q.N + g.bn - 1) / g.bn;
      g.tile_start = total_pair;
      total_pair += g.tiles_m * g.tiles_n;
      if (!make_tmap(&g.tmA, q.A, q.M, q.K, q.lda, TC_BM)) return EPARA_E_CUDA;
      if (!make_tmap(&g.tmW, q.W, q.N, q.K, q.ldw, g.bn / 2)) return EPARA_E_CUDA;
      if (!make_tmap_c(&g.tmC, q.C, q.M, q.N, q.ldc, q.epilogue)) return EPARA_E_CUDA;
      gs_pair.push_back(g);
      continue;
    }
    const int tm = simt ? SIMT_TILE : TC_BM, tn = simt ? SIMT_TILE : g.bn;
    g.tiles_m = (q.M + tm - 1) / tm; g.tiles_n = (q.N + tn - 1) / tn;
    g.tile_start = total;
    total += g.tiles_m * g.tiles_n * g.ksplit;
    if (!simt && q.M > 0) {
      if (!make_tmap(&g.tmA, q.A, q.M, q.K, q.lda, TC_BM)) return EPARA_E_CUDA;
      if (!make_tmap(&g.tmW, q.W, q.N, q.K, q.ldw, g.bn)) return EPARA_E_CUDA;
      if (!make_tmap_c(&g.tmC, q.C, q.M, q.N, q.ldc, q.epilogue)) return EPARA_E_CUDA;
    }
    if (g.ksplit > 1) {
      soff = align_up(soff, 256);
      g.partial = (float*)((unsigned char*)scratch + soff);
      soff += (size_t)g.ksplit * g.tiles_m * TC_BM * g.tiles_n * g.bn * 4;
      soff = align_up(soff, 256);
      g.counters = (int*)((unsigned char*)scratch + soff);
      if (cudaMemsetAsync(g.counters, 0, (size_t)g.tiles_m * g.tiles_n * sizeof(int), st) != cudaSuccess) return EPARA_E_CUDA;
      soff += (size_t)g.tiles_m * g.tiles_n * sizeof(int);
    }
    gs.push_back(g);
  }
  int* status = (int*)scratch;
  GemmGroup* dev_groups = (GemmGroup*)((unsigned char*)scratch + 256);
  GemmGroup* dev_stream = dev_groups + gs.size();
  GemmGroup* dev_pair = dev_stream + gs_stream.size();
  GemmGroup* dev_swap[4];
  dev_swap[0] = dev_pair + gs_pair.size();
  for (int i = 1; i < 4; ++i) dev_swap[i] = dev_swap[i - 1] + gs_swap[i - 1].size();
  for (int i = 0; i < 4; ++i)
    if (!gs_swap[i].empty() &&
        cudaMemcpyAsync(dev_swap[i], gs_swap[i].data(), gs_swap[i].size() * sizeof(GemmGroup), cudaMemcpyHostToDevice, st) != cudaSuccess)
      return EPARA_E_CUDA;
  if (cudaMemsetAsync(status, 0, 256, st) != cudaSuccess) return EPARA_E_CUDA;
  // (a copy from pageable host memory is staged before cudaMemcpyAsync returns, so the vectors may go out of scope)
  if (!gs.empty() &&
      cudaMemcpyAsync(dev_groups, gs.data(), gs.size() * sizeof(GemmGroup), cudaMemcpyHostToDevice, st) != cudaSuccess)
    return EPARA_E_CUDA;
  if (!gs_stream.empty() &&
      cudaMemcpyAsync(dev_stream, gs_stream.data(), gs_stream.size() * sizeof(GemmGroup), cudaMemcpyHostToDevice, st) != cudaSuccess)
    return EPARA_E_CUDA;
  if (!gs_pair.empty() &&
      cudaMemcpyAsync(dev_pair, gs_pair.data(), gs_pair.size() * sizeof(GemmGroup), cudaMemcpyHostToDevice, st) != cudaSuccess)
    return EPARA_E_CUDA;
  cudaError_t err = cudaSuccess;
  if (simt) {
    launch_gemm_simt(dev_groups, (int)gs.size(), total, st);
    err = cudaGetLastError();
  } else {
    const int sm = sm_count;
    int max_bn = 0;
    for (const GemmGroup& g : gs) max_bn = std::max(max_bn, g.bn);
    err = launch_gemm_tc(dev_groups, (int)gs.size(), total, max_bn, status, sm, st);
    if (err == cudaSuccess)
      err = launch_gemm_stream(dev_stream, (int)gs_stream.size(), total_stream, max_rows_stream, st);
    if (err == cudaSuccess)
      err = launch_gemm_tc_pair(dev_pair, (int)gs_pair.size(), total_pair, status, sm, st);
    for (int i = 0; i < 4 && err == cudaSuccess; ++i)
      err = launch_gemm_swap(dev_swap[i], (int)gs_swap[i].size(), total_swap[i], 1 << i, status, sm, st);
  }
  return err == cudaSuccess ? EPARA_OK : EPARA_E_CUDA;
}

size_t epara_decode_attention_scratch_bytes(int B, int Hq, int hd, int max_len) {
  const int chunks = (max_len + ATTN_CHUNK - 1) / ATTN_CHUNK;
  return 256 + align_up((size_t)B * sizeof(AttnReq), 256) + align_up((size_t)B * Hq * chunks * (hd + 2) * 4, 256) +
         (size_t)B * Hq * sizeof(int);
}

int epara_decode_attention(int device, void* cuda_stream, const void* q, int q_stride, const void* kv_layer,
                           long long kv_pages, const int32_t* kv_lens, const int32_t* tables, int table_stride, void* out,
                           int B, int Hq, int Hkv, int hd, int max_len, void* scratch, size_t scratch_bytes) {
  if (!q || !kv_layer || !kv_lens || !tables || !out || !scratch || B < 0 || Hkv <= 0 || Hq % Hkv || max_len <= 0 ||
      kv_pages <= 0)
    return EPARA_E_INVALID;
  if ((reinterpret_cast<uintptr_t>(q) & 15) || (reinterpret_cast<uintptr_t>(kv_layer) & 15) || (q_stride % 8) ||
      (reinterpret_cast<uintptr_t>(scratch) & 255))
    return EPARA_E_INVALID;
  if (scratch_bytes < epara_decode_attention_scratch_bytes(B, Hq, hd, max_len)) return EPARA_E_RESOURCE;
  if (B == 0) return EPARA_OK;
  if (cudaSetDevice(device) != cudaSuccess) return EPARA_E_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  unsigned char* s = (unsigned char*)scratch;
  static_assert(sizeof(AttnDecGroup) <= DEC_STATUS_OFFSET && DEC_STATUS_OFFSET + sizeof(int) <= 256, "scratch header");
  AttnDecGroup g;
  memset(&g, 0, sizeof(g));
  const int g_chunks = (max_len + ATTN_CHUNK - 1) / ATTN_CHUNK;
  AttnReq* reqs = (AttnReq*)(s + 256);
  g.q = (const bf16*)q; g.q_stride = q_stride; g.kv_layer = (const bf16*)kv_layer; g.reqs = reqs; g.out = (bf16*)out;
  g.partial = (float*)(s + 256 + align_up((size_t)B * sizeof(AttnReq), 256));
  g.counters = (int*)((unsigned char*)g.partial + align_up((size_t)B * Hq * g_chunks * (hd + 2) * 4, 256));
  g.B = B; g.Hq = Hq; g.Hkv = Hkv; g.hd = hd; g.max_chunks = g_chunks; g.req_start = 0;
  g.status = (int*)(s + DEC_STATUS_OFFSET);
  g.kv_pages = kv_pages;
  // one set-up kernel writes the descriptor, clears the status word and the counters and fills the request table
  launch_attn_prepare(g, (AttnDecGroup*)s, reqs, kv_lens, tables, table_stride, max_len, B * Hq, st);
  cudaError_t e = launch_attn_decode((const AttnDecGroup*)s, 1, B, Hkv, Hq, g.max_chunks, hd, Hq / Hkv,
                                     attn_decode_fused(B, Hkv, g.max_chunks, device_sm_count(device)) ? 1 : 0, st);
  if (e == cudaErrorInvalidValue) return EPARA_E_UNSUPPORTED;
  return e == cudaSuccess ? EPARA_OK : EPARA_E_CUDA;
}

}  // extern "C"
