// Device-visible descriptors written by the host step planner and read by the kernels.
// One step uploads one blob holding the request table and, per launch, an array of groups
// (one group = one model's problem in that launch).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace epara {

typedef __nv_bfloat16 bf16;

enum : int { EPI_BIAS = 1, EPI_GELU = 2, EPI_SWIGLU = 4, EPI_RESID_F32 = 8 };

// Codes a kernel leaves in the step's device status word (0 = none).  1..49 are bounded waits that ran
// out (the role that gave up); the others are indices found out of range, whose access was skipped.
enum : int { ERR_PAGE_APPEND = 101, ERR_PAGE_ATTEND = 102, ERR_SELFTEST_WAIT = 90 };

// Per admitted request (model order, then batch order).
struct ReqDesc {
  const void* input;     // MLP row / ViT image
  const int32_t* table;  // decoder block table
  void* out_logits;
  int32_t* out_argmax;
  int token;             // decoder, single-token request: the token being decoded
  int kv_len;            // cached tokens before this step
  int n_blocks;
  int row_start;         // decoder: first activation row of the request (a prompt chunk takes n_tok rows)
  int n_tok;             // decoder: tokens of the request in this step (1 = decode, > 1 = prompt chunk)
  int pad[3];
};

// Decoder activations have one row per token.  Row r belongs to request `req`, sits at position `pos` of
// its sequence and holds token id `token`.
struct RowDesc {
  int req, pos, token, pad;
};

// C = epi(A W^T + bias).  tmA/tmW are the TMA maps of A [rows, K] and W [N, K] (K innermost,
// 128-byte swizzle, box 64 x 128 rows for A and 64 x bn rows for W).  The tensor-core kernel cuts
// the group into tiles_m x tiles_n tiles of 128 x bn and every tile into ksplit ranges of
// k-blocks; with ksplit > 1 each range leaves an fp32 partial in `partial` and the range that
// arrives last (counted in `counters`) adds them in range order and runs the epilogue.
struct alignas(64) GemmGroup {
  CUtensorMap tmA;
  CUtensorMap tmW;
  CUtensorMap tmC;   // output, written by TMA from the epilogue's staging rows: bf16 [rows, N] with a
                     // 32 x 32 box (SwiGLU: [rows, N/2], 16 x 32), or fp32 [rows, N] with a 16 x 32 box
                     // for the residual update (TMA reduce-add)
  const bf16* A;
  const bf16* W;
  void* C;
  const bf16* bias;
  int M, N, K;
  int lda, ldw, ldc;
  int epi;
  int tile_start;  // first work item of this group in the launch
  int tiles_m, tiles_n;
  int bn, ksplit;  // tensor-core kernel only: tile width (128 or 256), k ranges per tile
  float* partial;  // [ksplit][tiles_m * 128][tiles_n * bn] fp32, ksplit > 1 only
  int* counters;   // [tiles_m * tiles_n], zero between launches
  int c_rows;      // row extent of tmC (rows at and beyond it are never written)
  int stream;      // 1: at most 16 rows ever, runs in the weight-streaming kernel (16 W rows per block,
                   // tiles_n = ceil(N / 16), no TMA maps); 0: one-CTA tensor-core tiles; 2: 256-row tiles on
                   // CTA pairs (tiles_m counts 256-row tiles and tmW's box holds bn / 2 rows)
  int pad1, pad2;
};

struct GemmLaunch {      // header followed by groups
  int n_groups;
  int total_tiles;
};

enum : int { NORM_LN = 0, NORM_RMS = 1 };
struct NormGroup {
  const float* x;        // fp32 [M rows, row stride x_stride]
  bf16* y;               // bf16 [M, d]
  const bf16* gamma;
  const bf16* beta;      // LN only
  const int* row_index;  // when set, output row m reads input row row_index[m] (a decoder's last-token rows)
  long long x_stride;
  int M, d, kind;
  float eps;
};

enum : int { GATHER_ROWS = 0, GATHER_EMB = 1, GATHER_PATCH = 2 };
struct GatherGroup {
  const ReqDesc* reqs;
  const RowDesc* rows;   // EMB: one entry per output row
  void* out;             // ROWS: bf16 [B, ld]; EMB: fp32 [rows, d]; PATCH: bf16 [B*np, 3*p*p]
  const bf16* emb;       // EMB
  int kind, B, width, ld;
  int img, patch;
  int blocks;            // blocks this group needs
  int pad;
};

struct RopeGroup {
  bf16* qkv;             // [rows, (Hq+2Hkv)*hd], q rotated in place
  bf16* kv_layer;        // [pages][2][Hkv][16][hd]
  const ReqDesc* reqs;
  const RowDesc* rows;   // one entry per token row; B counts rows
  const float2* cs;      // [max position + 1][hd/2]: (cos, sin) of position * 10000^(-2j/hd)
  int* status;           // device word: set to ERR_PAGE_APPEND when a block table names a page outside the pool
  long long kv_pages;    // pages of the pool; a page id outside [0, kv_pages) is reported, its write skipped
  int B, Hq, Hkv, hd;
};

struct AttnReq {
  const int32_t* table;
  int len;               // tokens to attend (cached + appended)
  int row;               // activation row of the request's token (q is read and the output written there)
};

// Causal attention of prompt chunks (one layer): request i has n_tok query tokens in rows row_start ..,
// token t at position kv_len + t attends to positions 0 .. kv_len + t of its paged cache (the chunk's own
// k, v were appended by the kernel before).  One block per (request, query head, tile of 64 tokens).
struct PrefillReq {
  const int32_t* table;
  int row_start, n_tok, kv_len;
  int blk_start;         // first block of this request within its group
};
struct AttnPrefillGroup {
  const bf16* qkv;       // [rows, q_stride], query head h at column h*hd
  const bf16* kv_layer;
  const PrefillReq* reqs;
  bf16* out;             // [rows, Hq*hd]
  int* status;
  long long kv_pages;
  int q_stride;
  int n_reqs, Hq, Hkv, hd;
  int blk_start;         // first block of this group in the launch
  int n_blocks;
};

struct AttnDecGroup {
  const bf16* q;         // [B, q_stride], head h at column h*hd
  const bf16* kv_layer;
  const AttnReq* reqs;
  bf16* out;             // [B, Hq*hd]
  float* partial;        // [B][Hq][max_chunks][hd + 2]  (m, l, o[hd]); requests of more than one chunk
  int* counters;         // [B][Hkv] chunks that have arrived; zero between launches
  int q_stride;
  int B, Hq, Hkv, hd;
  int max_chunks;
  int req_start;         // first grid.z index of this group
  int reqs_stable;       // 1: `reqs` was uploaded before the step's first kernel (a block past a request's
                         // length may leave without the dependency wait); 0: an earlier kernel writes it
  int* status;           // device word: set to ERR_PAGE_ATTEND when a block table names a page outside the pool
  long long kv_pages;    // pages of the pool; a page id outside [0, kv_pages) is reported and read as absent
};

struct alignas(64) AttnEncGroup {
  CUtensorMap tmQ;       // tensor-core kernel: qkv [rows, 3d] bf16, box 64 columns x 128 rows, 128-byte swizzle
  CUtensorMap tmKV;      // same matrix, box 64 columns x KP rows
  const bf16* qkv;       // [B*T, 3d]: q | k | v, head h at column h*hd within each
  bf16* out;             // [B*T, d]
  int B, T, H, hd;
  int blk_start;         // first block (item) of this group
  int q_blocks;          // query blocks per (image, head); 1 for the tensor-core kernel
  int tc;                // 1: runs in the tensor-core kernel (hd 64, T <= ENC_TC_MAX_T), fixed when the model is placed
  int KP;                // T rounded up to a multiple of 16
  int pad[8];
};

// One transformer MLP block of an encoder as a single work unit of the fused kernel:
// z += GELU(h W1^T + b1) W2^T + b2 with h bf16 [rows, d], W1 [F, d], W2 [d, F], z fp32 [rows, d].
// d is a multiple of 64 and at most 384 (the output accumulator of a 128-row tile must fit the tensor memory
// beside one 128-column chunk of the hidden layer), F a multiple of 128.
struct alignas(64) MlpGroup {
  CUtensorMap tmX;       // h [rows, d] bf16, box 64 columns x 128 rows, 128-byte swizzle
  CUtensorMap tmW1;      // W1 [F, d] bf16, box 64 x 64 rows (one CTA of a pair loads half of a chunk's 128 rows)
  CUtensorMap tmW2;      // W2 [d, F] bf16, box 64 x n2/2 rows (n2 = d, or d / 2 when d > 256: two MMAs per k step)
  CUtensorMap tmC;       // z [rows, d] fp32, box 16 columns x 32 rows (TMA reduce-add of the epilogue)
  const bf16* b1;        // [F] or null
  const bf16* b2;        // [d] or null
  int M, d, F;
  int tile_start;        // first work item (256-row tile) of this group in the launch
  int tiles_m;
  int c_rows;            // row extent of tmC
  int pad[8];
};

struct AssembleGroup {   // z[b, 0] = cls + pos[0]; z[b, 1+p] = E[b*np + p] + pos[1+p]
  const bf16* E;
  const bf16* cls;
  const bf16* pos;
  float* z;
  int B, T, d, pad;
};

struct OutputGroup {     // copy logits rows to the requests' buffers and take the argmax
  const bf16* logits;    // [B, ld]
  const ReqDesc* reqs;
  int B, N, ld, pad;
};

}  // namespace epara

// Group arrays are packed back to back in the step blob: sizes must keep 8-byte alignment.
namespace epara {
static_assert(sizeof(GemmGroup) % 64 == 0, "GemmGroup holds 64-byte aligned TMA maps");
static_assert(sizeof(AttnPrefillGroup) % 8 == 0 && sizeof(PrefillReq) % 8 == 0 && sizeof(RowDesc) == 16, "descriptor sizes");
static_assert(sizeof(NormGroup) % 8 == 0 && sizeof(GatherGroup) % 8 == 0 && sizeof(RopeGroup) % 8 == 0 &&
              sizeof(AttnDecGroup) % 8 == 0 && sizeof(AttnEncGroup) % 64 == 0 && sizeof(MlpGroup) % 64 == 0 && sizeof(AssembleGroup) % 8 == 0 &&
              sizeof(OutputGroup) % 8 == 0 && sizeof(ReqDesc) % 16 == 0 && sizeof(AttnReq) % 16 == 0,
              "descriptor sizes");
}  // namespace epara
