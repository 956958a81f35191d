// Host-side launchers of the step's kernels.  `groups` pointers are device memory.
#pragma once
#include <cuda_runtime.h>
#include "desc.h"

namespace epara {

constexpr int GATHER_PATCH_ROWS = 8;   // patch rows per block of the patch gather
void launch_gather(const GatherGroup* groups, int n_groups, int max_blocks, cudaStream_t st);
int norm_blocks(int M, int d);
void launch_norm(const NormGroup* groups, int n_groups, int max_blocks, cudaStream_t st);
void launch_rope_append(const RopeGroup* groups, int n_groups, int max_B, cudaStream_t st);
void launch_assemble(const AssembleGroup* groups, int n_groups, int max_rows, cudaStream_t st);
void launch_output(const OutputGroup* groups, int n_groups, int max_B, cudaStream_t st);

// Plain CUDA-core grouped GEMM, 64 x 64 tiles (comparator for the tensor-core kernel).
constexpr int SIMT_TILE = 64;
void launch_gemm_simt(const GemmGroup* groups, int n_groups, int total_tiles, cudaStream_t st);

// tcgen05 grouped GEMM, 128 x bn tiles (bn = 128 or 256 per group), persistent.  `status` is a
// device int the kernel sets non-zero if a bounded wait ran out.  total_items = sum over groups of
// tiles_m * tiles_n * ksplit.  Returns the cudaError of the launch configuration.
constexpr int TC_BM = 128;
constexpr int TC_BN_MAX = 256;
constexpr int TC_BK = 64;
void gemm_tc_config(long long rows_cap, int N, int K, int epi, int sm_count, int* bn, int* ksplit);
bool gemm_tc_pair_eligible(long long rows_cap, int N, int K, int epi, int bn, int ksplit);
bool gemm_mlp_eligible(long long rows_cap, int d, int F);
cudaError_t launch_gemm_mlp_pair(const MlpGroup* groups, int n_groups, int total_items, int* status, int sm_count,
                                 cudaStream_t st);
cudaError_t launch_gemm_tc_pair(const GemmGroup* groups, int n_groups, int total_items, int* status, int sm_count,
                                cudaStream_t st);
cudaError_t launch_gemm_tc(const GemmGroup* groups, int n_groups, int total_items, int max_bn, int* status,
                           int sm_count, cudaStream_t st);   // max_bn: widest tile among the groups

// Swapped-operand tensor-core GEMM for groups of 17 to 128 rows (GemmGroup::stream == 3): a cluster of `ksplit`
// CTAs per tile of 128 output columns; all groups of a launch share ksplit.  GemmGroup::bn holds the row capacity
// rounded up to 16, tmW the weight map (box 128 rows), tmA the activation map (box bn rows); tile_start counts
// tiles.  total_items = sum of gemm_swap_tiles(N).
int gemm_swap_ksplit(int N, int K, int sm_count);
int gemm_swap_tiles(int N);
cudaError_t launch_gemm_swap(const GemmGroup* groups, int n_groups, int total_items, int ksplit, int* status, int sm_count,
                             cudaStream_t st);
constexpr int GEMM_SWAP_MAX_ROWS = 128;

// Weight-streaming GEMM for groups that never exceed 16 rows (GemmGroup::stream): one block per 16
// rows of W over the whole K, mma.sync, no tensor maps.  total_items = sum of gemm_stream_tiles(N).
constexpr int GEMM_STREAM_MAX_ROWS = 16;
int gemm_stream_tiles(int N);
cudaError_t launch_gemm_stream(const GemmGroup* groups, int n_groups, int total_items, int max_rows, cudaStream_t st);

// Decode attention, split-KV over 256-token chunks.  fused = 1: the block of a (request, kv head) that
// finishes last merges the chunk partials (AttnDecGroup::counters must be zero at launch and is left
// zero); fused = 0: a second kernel merges them.  attn_decode_fused() is the rule that picks the mode
// from the launch's block count; both modes give the same bits.
constexpr int ATTN_CHUNK = 256;
bool attn_decode_fused(int total_B, int max_Hkv, int max_chunks, int sm_count);
cudaError_t launch_attn_decode(const AttnDecGroup* groups, int n_groups, int total_B, int max_Hkv, int max_Hq,
                               int max_chunks, int hd, int gqa, int fused, cudaStream_t st);
// Set-up of a single-kernel decode-attention call on the stream: writes `g` to `dst`, clears *g.status and
// g.counters[0 .. n_counters), fills reqs[b] = {tables + b*stride, kv_lens[b] clamped to [0, max_len]}.
void launch_attn_prepare(const AttnDecGroup& g, AttnDecGroup* dst, AttnReq* reqs, const int32_t* kv_lens,
                         const int32_t* tables, int stride, int max_len, int n_counters, cudaStream_t st);
constexpr int DEC_STATUS_OFFSET = 192;   // byte offset of the status word in a single-kernel call's scratch

// Causal attention of prompt chunks (head size 64 or 128), one block per (request, query head, 64 query tokens).
constexpr int PREFILL_TILE = 64;
inline int attn_prefill_blocks(int n_tok, int Hq) { return (n_tok + PREFILL_TILE - 1) / PREFILL_TILE * Hq; }
cudaError_t launch_attn_prefill(const AttnPrefillGroup* groups, int n_groups, int total_blocks, int hd, cudaStream_t st);

// Encoder attention on tcgen05 for groups with AttnEncGroup::tc (hd 64, T <= ENC_TC_MAX_T): persistent,
// one item per (image, head); total_items = sum of B * H.  `status` as for the GEMM.
constexpr int ENC_TC_MAX_T = 224;
cudaError_t launch_attn_encoder_tc(const AttnEncGroup* groups, int n_groups, int total_items, int* status, int sm_count,
                                   cudaStream_t st);

// Encoder (bidirectional) attention on mma.sync, one block per (image, head, query block).
cudaError_t launch_attn_encoder(const AttnEncGroup* groups, int n_groups, int total_blocks, int max_T,
                                cudaStream_t st);
int attn_encoder_q_blocks(int T);

}  // namespace epara
