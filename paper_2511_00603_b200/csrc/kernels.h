// Host-side launchers of the step's kernels.  `groups` pointers are device memory.
#pragma once
#include <cuda_runtime.h>
#include "desc.h"

namespace epara {

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
cudaError_t launch_gemm_tc(const GemmGroup* groups, int n_groups, int total_items, int* status, int sm_count,
                           cudaStream_t st);

// Decode attention (split-KV over 256-token chunks) and the combine of the chunk partials.
constexpr int ATTN_CHUNK = 256;
cudaError_t launch_attn_decode(const AttnDecGroup* groups, int n_groups, int total_B, int max_Hkv, int max_chunks,
                               int hd, int gqa, cudaStream_t st);
cudaError_t launch_attn_combine(const AttnDecGroup* groups, int n_groups, int total_B, int max_Hq, int hd,
                                cudaStream_t st);
// Fills AttnReq[b] = {tables + b*stride, kv_lens[b]} on the device.
void launch_attn_fill_reqs(AttnReq* reqs, const int32_t* kv_lens, const int32_t* tables, int stride, int B,
                           cudaStream_t st);

// Encoder (bidirectional) attention, one block per (image, head, query block).
cudaError_t launch_attn_encoder(const AttnEncGroup* groups, int n_groups, int total_blocks, int max_T,
                                cudaStream_t st);
int attn_encoder_q_blocks(int T);

}  // namespace epara
