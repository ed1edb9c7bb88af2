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
  int* status;                // device status word
};

// KV position (among the subnet's kept groups) that kept head hq of subnet s reads.  The two index arrays are
// checked on the way: an entry outside its range is replaced by 0 (so that nothing is read or written out of
// bounds) and TWIST_ERR_BAD_INDEX is recorded in the status word.
__device__ inline int kv_position(const AttnParams& p, int s, int hq) {
  if (!p.head_idx) return hq;
  int g = p.head_idx[(long long)s * p.heads + hq] / p.per_group;
  if ((unsigned)g >= (unsigned)p.n_kv_heads) { atomicMin(p.status, (int)TWIST_ERR_BAD_INDEX); g = 0; }
  int pos = p.kv_pos[(long long)s * p.n_kv_heads + g];
  if ((unsigned)pos >= (unsigned)p.kv_max) { atomicMin(p.status, (int)TWIST_ERR_BAD_INDEX); pos = 0; }
  return pos;
}


// Tensor-core kernels (d_head = 64), defined in attn_core_tc.cu.  The backward expects delta to be filled.
int attn_fwd_tc(const AttnParams& p, int n_subnets, cudaStream_t st);
int attn_bwd_tc(const AttnParams& p, int n_subnets, cudaStream_t st);

}  // namespace twist
