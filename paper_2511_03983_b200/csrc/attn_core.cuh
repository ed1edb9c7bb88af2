// Parameters shared by the attention-core kernels (fp32 SIMT kernels in attn_core.cu, tensor-core kernels in
// attn_core_tc.cu).
#pragma once
#include "common.cuh"

namespace twist {

struct AttnParams {
  const __nv_bfloat16* qkv;   // [S][T][nq]
  __nv_bfloat16* out;         // [S][T][a_sub]
  float* lse;                 // [S][H'][T]   natural-log sum of exp(scores)
  const __nv_bfloat16* d_out; // [S][T][a_sub]
  __nv_bfloat16* d_qkv;       // [S][T][nq]
  float* delta;               // [S][H'][T]   rowsum(dA * A)
  const int32_t* head_idx;    // [S][H'] kept head ids, or null (no KV sharing: head hq reads KV position hq)
  const int32_t* kv_pos;      // [S][H_kv] position of a KV group among the subnet's kept groups
  const int32_t* kv_count;    // [S] kept KV groups, or null (= kv_max)
  int n_seqs, seq_len, heads, kv_max, d_head, per_group, n_kv_heads;
  int a_sub, nq, T;
  float scale_log2;           // log2(e) / sqrt(d_head)
};


// Tensor-core kernels (d_head = 64), defined in attn_core_tc.cu.  The backward expects delta to be filled.
int attn_fwd_tc(const AttnParams& p, int n_subnets, cudaStream_t st);
int attn_bwd_tc(const AttnParams& p, int n_subnets, cudaStream_t st);

}  // namespace twist
