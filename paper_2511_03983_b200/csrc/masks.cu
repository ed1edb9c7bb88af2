// twist_sample_masks / twist_kv_groups: subnet generator (Algorithm 1, "Generate Training Subnet
// Blueprint") as integer-only kernels.  One CTA builds one row A[s] of one layer's blueprint:
//   flags <- common blocks; deal a seeded random order of the non-common blocks round-robin
//   (block i of the order goes to subnet i mod S); fill with the N_empty smallest fill keys among
//   the blocks the subnet lacks; emit the kept blocks in ascending order (warp ballot/popc scan).
// Random order = ascending 64-bit keys (48 hash bits | 16-bit block id), sorted in shared memory.
#include "common.cuh"

namespace twist {
namespace {

constexpr uint64_t kGolden = 0x9E3779B97F4A7C15ull;

__host__ __device__ inline uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// Counter hash of (seed, round, layer, kind, stream, subnet); block keys derive from it.
__device__ inline uint64_t stream_base(uint64_t seed, uint64_t rnd, int layer, int kind, int stream, int s) {
  uint64_t h = mix64(seed + kGolden);
  h = mix64(h + rnd);
  h = mix64(h + (uint64_t)(((uint32_t)layer << 16) | ((uint32_t)kind << 8) | (uint32_t)stream));
  return mix64(h + (uint64_t)s);
}

__device__ inline uint64_t block_key(uint64_t base, int b) {
  return (mix64(base + (uint64_t)b) & ~0xFFFFull) | (uint64_t)b;
}

struct CommonList {
  int32_t n;
  int32_t id[TWIST_MAX_COMMON];
};

// Ascending bitonic sort of np (power of two) keys in shared memory by the whole CTA.
__device__ void bitonic_sort(uint64_t* keys, int np) {
  for (int k = 2; k <= np; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int i = threadIdx.x; i < np; i += blockDim.x) {
        int ixj = i ^ j;
        if (ixj > i) {
          uint64_t a = keys[i], b = keys[ixj];
          bool asc = (i & k) == 0;
          if ((a > b) == asc) { keys[i] = b; keys[ixj] = a; }
        }
      }
      __syncthreads();
    }
  }
}

// Sum of v over the CTA (all threads get the result).  scratch: 33 ints of shared memory.
__device__ int block_sum(int v, int* scratch) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  if (warp == 0) {
    int t = lane < nw ? scratch[lane] : 0;
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (lane == 0) scratch[32] = t;
  }
  __syncthreads();
  return scratch[32];
}

__global__ void sample_rows_kernel(uint64_t seed, uint64_t rnd, int layer_begin, int kind, int n_full, int S,
                                   int n_sub, int mode, int np, const __grid_constant__ CommonList common,
                                   int32_t* __restrict__ idx) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint64_t* keys = reinterpret_cast<uint64_t*>(smem_raw);
  int* scratch = reinterpret_cast<int*>(keys + np);               // 64 ints
  unsigned char* flags = reinterpret_cast<unsigned char*>(scratch + 64);   // n_full bytes
  const int s = blockIdx.x, layer = layer_begin + blockIdx.y;
  const int tid = threadIdx.x, nt = blockDim.x;

  for (int b = tid; b < n_full; b += nt) flags[b] = 0;
  __syncthreads();
  for (int i = tid; i < common.n; i += nt) flags[common.id[i]] = 1;             // step 1: common blocks
  __syncthreads();

  if (mode == TWIST_MODE_COVER) {                                                // step 2: round-robin deal
    const uint64_t base = stream_base(seed, rnd, layer, kind, 0, 0);
    for (int b = tid; b < np; b += nt)
      keys[b] = (b < n_full && !flags[b]) ? block_key(base, b) : ~0ull;
    __syncthreads();
    bitonic_sort(keys, np);
    const int n_noncommon = n_full - common.n;
    for (int i = tid; i < n_noncommon; i += nt)
      if (i % S == s) flags[keys[i] & 0xFFFFull] = 1;
    __syncthreads();
  }

  int local = 0;                                                                 // step 3: fill
  for (int b = tid; b < n_full; b += nt) local += flags[b];
  const int n_empty = n_sub - block_sum(local, scratch);
  if (n_empty > 0) {
    const uint64_t base = stream_base(seed, rnd, layer, kind, 1, s);
    for (int b = tid; b < np; b += nt)
      keys[b] = (b < n_full && !flags[b]) ? block_key(base, b) : ~0ull;
    __syncthreads();
    bitonic_sort(keys, np);
    for (int i = tid; i < n_empty; i += nt) flags[keys[i] & 0xFFFFull] = 1;
    __syncthreads();
  }

  // step 4: emit kept blocks in ascending order.  Each warp owns a contiguous range of blocks;
  // ballot + popc ranks the kept blocks inside each 32-block group.
  const int nw = nt >> 5, warp = tid >> 5, lane = tid & 31;
  const int per_warp = ((n_full + nw - 1) / nw + 31) & ~31;
  const int b0 = warp * per_warp, b1 = min(n_full, b0 + per_warp);
  int cnt = 0;
  for (int bb = b0; bb < b1; bb += 32) {   // bb is warp-uniform
    const int b = bb + lane;
    cnt += __popc(__ballot_sync(0xffffffffu, b < b1 && flags[b]));
  }
  // exclusive scan of the per-warp counts
  __syncthreads();
  if (lane == 0) scratch[warp] = cnt;
  __syncthreads();
  int offset = 0;
  for (int w = 0; w < warp; ++w) offset += scratch[w];
  int32_t* out = idx + ((size_t)blockIdx.y * S + s) * n_sub;
  for (int bb = b0; bb < b1; bb += 32) {
    int b = bb + lane;
    bool keep = b < b1 && flags[b];
    unsigned m = __ballot_sync(0xffffffffu, keep);
    if (keep) {
      int r = offset + __popc(m & ((1u << lane) - 1u));
      if (r < n_sub) out[r] = b;
    }
    offset += __popc(m);
  }
}

// cover[l][b] and pos[l][s][b] from the sorted rows: binary search of b in every row.
__global__ void cover_pos_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ count, int n_full, int S,
                                 int row_len, uint32_t* __restrict__ cover, int32_t* __restrict__ pos) {
  const int l = blockIdx.y;
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= n_full) return;
  uint32_t mask = 0;
  for (int s = 0; s < S; ++s) {
    const int32_t* row = idx + ((size_t)l * S + s) * row_len;
    int n = count ? count[l * S + s] : row_len;
    int lo = 0, hi = n;
    while (lo < hi) {
      int mid = (lo + hi) >> 1;
      if (row[mid] < b) lo = mid + 1; else hi = mid;
    }
    bool hit = lo < n && row[lo] == b;
    pos[((size_t)l * S + s) * n_full + b] = hit ? lo : -1;
    if (hit) mask |= 1u << s;
  }
  cover[(size_t)l * n_full + b] = mask;
}

// mask[s][r] = bit (subnet_begin + s) of cover[r / block_rows]
__global__ void hidden_mask_kernel(const uint32_t* __restrict__ cover, long long rows, int block_rows, int subnet_begin,
                                   int n_subnets, uint8_t* __restrict__ mask) {
  const long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= rows) return;
  const uint32_t c = cover[r / block_rows];
  for (int s = 0; s < n_subnets; ++s) mask[(long long)s * rows + r] = (uint8_t)((c >> (subnet_begin + s)) & 1u);
}

// One CTA per subnet: mask over the columns [Q heads | K groups | V groups] and the number of marked columns.
__global__ void qkv_col_mask_kernel(const uint32_t* __restrict__ head_cover, const uint32_t* __restrict__ kv_cover,
                                    int n_heads, int n_kv, int d_head, int subnet_begin, uint8_t* __restrict__ mask,
                                    int32_t* __restrict__ count) {
  const int s = blockIdx.x, bit = subnet_begin + s;
  const int width = (n_heads + 2 * n_kv) * d_head;
  for (int c = threadIdx.x; c < width; c += blockDim.x) {
    const int blk = c / d_head;
    const uint32_t cov = blk < n_heads ? head_cover[blk] : kv_cover[(blk - n_heads) % n_kv];
    mask[(long long)s * width + c] = (uint8_t)((cov >> bit) & 1u);
  }
  if (threadIdx.x == 0) {
    int n = 0;
    for (int h = 0; h < n_heads; ++h) n += (head_cover[h] >> bit) & 1u;
    for (int g = 0; g < n_kv; ++g) n += 2 * ((kv_cover[g] >> bit) & 1u);
    count[s] = n * d_head;
  }
}

// out[s][t][c] = mask[s][c] ? in[s][t][c] : 0 for bf16 activations, 8 columns (16 bytes) per thread.
__global__ void __launch_bounds__(256) apply_col_mask_kernel(const uint4* __restrict__ in, const uint8_t* __restrict__ mask,
                                                             uint4* __restrict__ out, long long vecs_per_subnet,
                                                             int vecs_per_row, long long total) {
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < total; v += (long long)gridDim.x * blockDim.x) {
    const long long s = v / vecs_per_subnet;
    const int c = (int)((v - s * vecs_per_subnet) % vecs_per_row);
    const uint2 m = *reinterpret_cast<const uint2*>(mask + (s * vecs_per_row + c) * 8);
    const uint4 x = in[v];
    uint4 y;
    y.x = (x.x & ((m.x & 0x000000FFu) ? 0x0000FFFFu : 0u)) | (x.x & ((m.x & 0x0000FF00u) ? 0xFFFF0000u : 0u));
    y.y = (x.y & ((m.x & 0x00FF0000u) ? 0x0000FFFFu : 0u)) | (x.y & ((m.x & 0xFF000000u) ? 0xFFFF0000u : 0u));
    y.z = (x.z & ((m.y & 0x000000FFu) ? 0x0000FFFFu : 0u)) | (x.z & ((m.y & 0x0000FF00u) ? 0xFFFF0000u : 0u));
    y.w = (x.w & ((m.y & 0x00FF0000u) ? 0x0000FFFFu : 0u)) | (x.w & ((m.y & 0xFF000000u) ? 0xFFFF0000u : 0u));
    out[v] = y;
  }
}

// One thread per (layer, subnet): kept KV groups of the sorted kept heads.
__global__ void kv_groups_kernel(const int32_t* __restrict__ head_idx, int total, int head_keep, int per_group,
                                 int n_kv, int d_head, int32_t* __restrict__ kv_idx, int32_t* __restrict__ kv_count,
                                 int32_t* __restrict__ kv_cols) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= total) return;
  const int32_t* row = head_idx + (size_t)t * head_keep;
  int32_t* out = kv_idx + (size_t)t * n_kv;
  int n = 0, last = -1;
  for (int j = 0; j < head_keep; ++j) {
    int g = row[j] / per_group;
    if (g != last) { out[n++] = g; last = g; }
  }
  kv_count[t] = n;
  kv_cols[t] = n * d_head;
  for (int j = n; j < n_kv; ++j) out[j] = -1;
}

}  // namespace
}  // namespace twist

extern "C" int32_t twist_sample_masks(uint64_t seed, uint64_t round, int32_t layer_begin, int32_t n_layers,
                                      int32_t kind, int32_t n_full, int32_t n_subnets, int32_t n_sub,
                                      const int32_t* common, int32_t n_common, int32_t sample_mode, int32_t* idx,
                                      uint32_t* cover, int32_t* pos, void* stream) {
  using namespace twist;
  if (!idx || !cover || !pos || (n_common > 0 && !common)) return TWIST_ERR_NULL;
  if (n_layers <= 0 || n_full <= 0 || n_subnets <= 0 || n_sub <= 0 || n_common < 0 || layer_begin < 0 ||
      (kind != TWIST_KIND_FFN && kind != TWIST_KIND_HEAD) ||
      (sample_mode != TWIST_MODE_COVER && sample_mode != TWIST_MODE_IID))
    return TWIST_ERR_SHAPE;
  if (n_full > TWIST_MAX_BLOCKS || n_subnets > TWIST_MAX_SUBNETS || n_common > TWIST_MAX_COMMON ||
      layer_begin + n_layers > 65536)
    return TWIST_ERR_UNSUPPORTED;
  CommonList cl;
  cl.n = n_common;
  for (int i = 0; i < n_common; ++i) {
    if (common[i] < 0 || common[i] >= n_full || (i > 0 && common[i] <= common[i - 1])) return TWIST_ERR_BAD_INDEX;
    cl.id[i] = common[i];
  }
  // size bound of Sec. 3.1
  if (n_sub > n_full || n_sub < n_common) return TWIST_ERR_INFEASIBLE;
  if (sample_mode == TWIST_MODE_COVER &&
      (int64_t)n_full - n_common > (int64_t)n_subnets * ((int64_t)n_sub - n_common))
    return TWIST_ERR_INFEASIBLE;

  int np = 32;
  while (np < n_full) np <<= 1;
  const int threads = np >= 4096 ? 1024 : 256;
  const size_t smem = (size_t)np * 8 + 64 * 4 + (size_t)n_full;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The shared-memory limit is raised once per device to what the largest block count needs: setting it per call
  // would let two host threads with different sizes lower it between one thread's set and its launch.
  static bool configured[64] = {false};
  const int slot = device_slot();
  if (!configured[slot]) {
    TWIST_CUDA_TRY(cudaFuncSetAttribute(sample_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        TWIST_MAX_BLOCKS * 8 + 64 * 4 + TWIST_MAX_BLOCKS));
    configured[slot] = true;
  }
  sample_rows_kernel<<<dim3(n_subnets, n_layers), threads, smem, st>>>(seed, round, layer_begin, kind, n_full,
                                                                       n_subnets, n_sub, sample_mode, np, cl, idx);
  TWIST_LAUNCH_CHECK();
  cover_pos_kernel<<<dim3((n_full + 255) / 256, n_layers), 256, 0, st>>>(idx, nullptr, n_full, n_subnets, n_sub,
                                                                         cover, pos);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

extern "C" int32_t twist_hidden_mask(const uint32_t* cover, int32_t n_full, int32_t block_rows, int32_t subnet_begin,
                                     int32_t n_subnets, uint8_t* mask, void* stream) {
  using namespace twist;
  if (!cover || !mask) return TWIST_ERR_NULL;
  if (n_full <= 0 || block_rows <= 0 || subnet_begin < 0 || n_subnets <= 0) return TWIST_ERR_SHAPE;
  if (subnet_begin + n_subnets > TWIST_MAX_SUBNETS) return TWIST_ERR_UNSUPPORTED;
  const long long rows = (long long)n_full * block_rows;
  hidden_mask_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      cover, rows, block_rows, subnet_begin, n_subnets, mask);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

extern "C" int32_t twist_qkv_col_mask(const uint32_t* head_cover, const uint32_t* kv_cover, int32_t n_heads,
                                      int32_t n_kv_heads, int32_t d_head, int32_t subnet_begin, int32_t n_subnets,
                                      uint8_t* mask, int32_t* count, void* stream) {
  using namespace twist;
  if (!head_cover || !kv_cover || !mask || !count) return TWIST_ERR_NULL;
  if (n_heads <= 0 || n_kv_heads <= 0 || d_head <= 0 || subnet_begin < 0 || n_subnets <= 0) return TWIST_ERR_SHAPE;
  if (subnet_begin + n_subnets > TWIST_MAX_SUBNETS) return TWIST_ERR_UNSUPPORTED;
  qkv_col_mask_kernel<<<n_subnets, 256, 0, static_cast<cudaStream_t>(stream)>>>(head_cover, kv_cover, n_heads, n_kv_heads,
                                                                              d_head, subnet_begin, mask, count);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

extern "C" int32_t twist_apply_col_mask(const void* in, const uint8_t* mask, void* out, int32_t n_subnets, int32_t tokens,
                                        int32_t width, void* stream) {
  using namespace twist;
  if (!in || !mask || !out) return TWIST_ERR_NULL;
  if (n_subnets <= 0 || tokens <= 0 || width <= 0 || width % 8 != 0) return TWIST_ERR_SHAPE;
  if (!aligned16(in) || !aligned16(out) || (reinterpret_cast<uintptr_t>(mask) & 7u)) return TWIST_ERR_SHAPE;
  const int vecs_per_row = width / 8;
  const long long per_subnet = (long long)tokens * vecs_per_row, total = per_subnet * n_subnets;
  long long blocks = (total + 255) / 256;
  const long long cap = (long long)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  apply_col_mask_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint4*>(in), mask, static_cast<uint4*>(out), per_subnet, vecs_per_row, total);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

extern "C" int32_t twist_kv_groups(const int32_t* head_idx, int32_t n_layers, int32_t n_subnets, int32_t head_keep,
                                   int32_t n_heads, int32_t n_kv_heads, int32_t d_head, int32_t* kv_idx,
                                   int32_t* kv_count, int32_t* kv_cols, uint32_t* kv_cover, int32_t* kv_pos,
                                   void* stream) {
  using namespace twist;
  if (!head_idx || !kv_idx || !kv_count || !kv_cols || !kv_cover || !kv_pos) return TWIST_ERR_NULL;
  if (n_layers <= 0 || n_subnets <= 0 || head_keep <= 0 || n_heads <= 0 || n_kv_heads <= 0 || d_head <= 0 ||
      n_heads % n_kv_heads != 0 || head_keep > n_heads)
    return TWIST_ERR_SHAPE;
  if (n_subnets > TWIST_MAX_SUBNETS) return TWIST_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int total = n_layers * n_subnets;
  kv_groups_kernel<<<(total + 127) / 128, 128, 0, st>>>(head_idx, total, head_keep, n_heads / n_kv_heads, n_kv_heads,
                                                        d_head, kv_idx, kv_count, kv_cols);
  TWIST_LAUNCH_CHECK();
  cover_pos_kernel<<<dim3((n_kv_heads + 255) / 256, n_layers), 256, 0, st>>>(kv_idx, kv_count, n_kv_heads, n_subnets,
                                                                             n_kv_heads, kv_cover, kv_pos);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}
