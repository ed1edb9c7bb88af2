// twist_gather_subnets (dispatcher, Sec. 3.2) and twist_aggregate (aggregator, Sec. 3.3).
// Both are HBM-bandwidth kernels: one warp moves one whole row with 16-byte accesses per lane,
// several independent loads in flight per lane, streaming stores.  Rows are >= 1.5 KB in every
// workload (8 KB at d_model = 4096 in bf16), so every access is fully coalesced.
#include "common.cuh"

namespace twist {
namespace {

struct GatherParams {
  twist_gather_segment seg[TWIST_MAX_SEGMENTS];
  long long row_end[TWIST_MAX_SEGMENTS];   // exclusive prefix end of each segment's rows (all subnets)
  int n_segs;
  int d;
  long long total_rows;
};

struct AggParams {
  twist_aggregate_segment seg[TWIST_MAX_SEGMENTS];
  long long row_end[TWIST_MAX_SEGMENTS];
  int n_segs;
  int d;
  int n_subnets;
  uint32_t live;
  long long total_rows;
};

__device__ inline uint4 ld_nc(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ inline void st_cs(uint4* p, uint4 v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ inline void st_cs2(uint2* p, uint2 v) {
  asm volatile("st.global.cs.v2.u32 [%0], {%1,%2};" :: "l"(p), "r"(v.x), "r"(v.y) : "memory");
}

__device__ inline uint4 widen_lo(uint4 v) {   // bf16 elements 0..3 of v -> 4 fp32 bit patterns
  return make_uint4(v.x << 16, v.x & 0xFFFF0000u, v.y << 16, v.y & 0xFFFF0000u);
}
__device__ inline uint4 widen_hi(uint4 v) {   // bf16 elements 4..7
  return make_uint4(v.z << 16, v.z & 0xFFFF0000u, v.w << 16, v.w & 0xFFFF0000u);
}

constexpr int kUnroll = 4;

// One warp per destination row.  ELEM = 2 (bf16) or 4 (fp32) bytes.
template <int ELEM>
__global__ void __launch_bounds__(256) gather_rows_kernel(const __grid_constant__ GatherParams p) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  const int chunks = p.d * ELEM / 16;                 // 16-byte chunks per row
  for (long long r = warp0; r < p.total_rows; r += nwarps) {
    int g = 0;
    while (g + 1 < p.n_segs && r >= p.row_end[g]) ++g;
    const twist_gather_segment& sg = p.seg[g];
    const long long rl = r - (g ? p.row_end[g - 1] : 0);
    const int rows_per_subnet = sg.n_keep * sg.block_rows;
    const int s = (int)(rl / rows_per_subnet);
    const int rem = (int)(rl - (long long)s * rows_per_subnet);
    const int j = rem / sg.block_rows, i = rem - j * sg.block_rows;
    const bool valid = sg.count ? (j < sg.count[s]) : true;
    const long long dst_row = sg.dst_row_offset + rem;
    uint4* dst = reinterpret_cast<uint4*>(static_cast<char*>(sg.dst) +
                                          ((long long)s * sg.dst_subnet_stride + dst_row * p.d) * ELEM);
    uint4* mst = sg.dst_master ? reinterpret_cast<uint4*>(sg.dst_master + (long long)s * sg.dst_subnet_stride +
                                                          dst_row * p.d)
                               : nullptr;
    const uint4* src = nullptr;
    if (valid) {
      const long long src_row = sg.src_row_offset + (long long)sg.idx[(long long)s * sg.idx_stride + j] * sg.block_rows + i;
      src = reinterpret_cast<const uint4*>(static_cast<const char*>(sg.src) + src_row * p.d * ELEM);
    }
    for (int c0 = lane; c0 < chunks; c0 += 32 * kUnroll) {
      uint4 v[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int c = c0 + 32 * u;
        v[u] = (valid && c < chunks) ? ld_nc(src + c) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int c = c0 + 32 * u;
        if (c < chunks) {
          st_cs(dst + c, v[u]);
          if (ELEM == 2 && mst) {
            st_cs(mst + 2 * c, widen_lo(v[u]));
            st_cs(mst + 2 * c + 1, widen_hi(v[u]));
          }
        }
      }
    }
  }
}

__device__ inline uint32_t pack_bf16x2_rn(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// One warp per full-model row: fp32 sum over the covering subnets in ascending order, IEEE divide.
template <bool BF16>
__global__ void __launch_bounds__(256) aggregate_rows_kernel(const __grid_constant__ AggParams p) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  const int chunks = p.d / 4;                          // float4 chunks per row
  for (long long r = warp0; r < p.total_rows; r += nwarps) {
    int g = 0;
    while (g + 1 < p.n_segs && r >= p.row_end[g]) ++g;
    const twist_aggregate_segment& sg = p.seg[g];
    const long long rl = r - (g ? p.row_end[g - 1] : 0);
    const int b = (int)(rl / sg.block_rows), i = (int)(rl - (long long)b * sg.block_rows);
    const uint32_t m = sg.cover[b] & p.live;
    if (m == 0) continue;                              // held by no live subnet: untouched
    const int cnt = __popc(m);
    const float4* mine = nullptr;                      // lane k holds the row pointer of the k-th covering subnet
    if (lane < cnt) {
      const int s = __fns(m, 0, lane + 1);
      const long long srow = sg.sub_row_offset + (long long)sg.pos[(long long)s * sg.n_full + b] * sg.block_rows + i;
      mine = reinterpret_cast<const float4*>(sg.sub + (long long)s * sg.sub_subnet_stride + srow * p.d);
    }
    const long long drow = sg.dst_row_offset + rl;
    const float denom = (float)cnt;
    for (int c0 = lane; c0 < chunks; c0 += 32 * kUnroll) {
      float4 acc[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int k = 0; k < cnt; ++k) {
        const float4* ptr = reinterpret_cast<const float4*>(__shfl_sync(0xffffffffu, (unsigned long long)mine, k));
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
          const int c = c0 + 32 * u;
          if (c < chunks) {
            uint4 raw = ld_nc(reinterpret_cast<const uint4*>(ptr + c));
            acc[u].x += __uint_as_float(raw.x);
            acc[u].y += __uint_as_float(raw.y);
            acc[u].z += __uint_as_float(raw.z);
            acc[u].w += __uint_as_float(raw.w);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int c = c0 + 32 * u;
        if (c < chunks) {
          float4 q = make_float4(acc[u].x / denom, acc[u].y / denom, acc[u].z / denom, acc[u].w / denom);
          uint4 qb = make_uint4(__float_as_uint(q.x), __float_as_uint(q.y), __float_as_uint(q.z), __float_as_uint(q.w));
          if (BF16) {
            if (sg.dst_f32) st_cs(reinterpret_cast<uint4*>(sg.dst_f32 + drow * p.d) + c, qb);
            st_cs2(reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(sg.dst) + drow * p.d) + c,
                   make_uint2(pack_bf16x2_rn(q.x, q.y), pack_bf16x2_rn(q.z, q.w)));
          } else {
            st_cs(reinterpret_cast<uint4*>(static_cast<float*>(sg.dst) + drow * p.d) + c, qb);
          }
        }
      }
    }
  }
}

int grid_for_rows(long long rows) {
  const long long warps_per_cta = 8;
  long long want = (rows + warps_per_cta - 1) / warps_per_cta;
  long long cap = (long long)sm_count() * 8;          // 8 resident CTAs of 256 threads per SM
  return (int)(want < cap ? (want > 0 ? want : 1) : cap);
}

}  // namespace
}  // namespace twist

extern "C" int32_t twist_gather_subnets(const twist_gather_segment* segs, int32_t n_segs, int32_t n_subnets,
                                        int32_t d, int32_t dtype, void* stream) {
  using namespace twist;
  if (!segs) return TWIST_ERR_NULL;
  if (n_segs <= 0 || n_segs > TWIST_MAX_SEGMENTS || n_subnets <= 0 || d <= 0) return TWIST_ERR_SHAPE;
  if (dtype != TWIST_FP32 && dtype != TWIST_BF16) return TWIST_ERR_SHAPE;
  const int elem = dtype == TWIST_BF16 ? 2 : 4;
  if ((d * elem) % 16 != 0) return TWIST_ERR_SHAPE;
  GatherParams p;
  memset(&p, 0, sizeof(p));
  long long total = 0;
  for (int g = 0; g < n_segs; ++g) {
    const twist_gather_segment& s = segs[g];
    if (!s.src || !s.dst || !s.idx) return TWIST_ERR_NULL;
    if (s.n_keep <= 0 || s.block_rows <= 0 || s.idx_stride < s.n_keep || s.src_row_offset < 0 ||
        s.dst_row_offset < 0 || s.dst_subnet_stride < 0 || (s.dst_subnet_stride * elem) % 16 != 0)
      return TWIST_ERR_SHAPE;
    if (!aligned16(s.src) || !aligned16(s.dst) || !aligned16(s.dst_master)) return TWIST_ERR_SHAPE;
    if (dtype == TWIST_FP32 && s.dst_master) return TWIST_ERR_UNSUPPORTED;   // an fp32 slice is its own master
    p.seg[g] = s;
    total += (long long)n_subnets * s.n_keep * s.block_rows;
    p.row_end[g] = total;
  }
  p.n_segs = n_segs;
  p.d = d;
  p.total_rows = total;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int grid = grid_for_rows(total);
  if (dtype == TWIST_BF16) gather_rows_kernel<2><<<grid, 256, 0, st>>>(p);
  else gather_rows_kernel<4><<<grid, 256, 0, st>>>(p);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

extern "C" int32_t twist_aggregate(const twist_aggregate_segment* segs, int32_t n_segs, int32_t n_subnets, int32_t d,
                                   int32_t dtype, uint32_t live_subnets, void* stream) {
  using namespace twist;
  if (!segs) return TWIST_ERR_NULL;
  if (n_segs <= 0 || n_segs > TWIST_MAX_SEGMENTS || n_subnets <= 0 || n_subnets > TWIST_MAX_SUBNETS || d <= 0)
    return TWIST_ERR_SHAPE;
  if (dtype != TWIST_FP32 && dtype != TWIST_BF16) return TWIST_ERR_SHAPE;
  if (d % 4 != 0 || (dtype == TWIST_BF16 && d % 8 != 0)) return TWIST_ERR_SHAPE;
  AggParams p;
  memset(&p, 0, sizeof(p));
  long long total = 0;
  for (int g = 0; g < n_segs; ++g) {
    const twist_aggregate_segment& s = segs[g];
    if (!s.dst || !s.sub || !s.cover || !s.pos) return TWIST_ERR_NULL;
    if (s.n_full <= 0 || s.block_rows <= 0 || s.dst_row_offset < 0 || s.sub_row_offset < 0 ||
        s.sub_subnet_stride < 0 || s.sub_subnet_stride % 4 != 0)
      return TWIST_ERR_SHAPE;
    if (!aligned16(s.dst) || !aligned16(s.sub) || !aligned16(s.dst_f32)) return TWIST_ERR_SHAPE;
    if (dtype == TWIST_FP32 && s.dst_f32) return TWIST_ERR_UNSUPPORTED;      // dst already is the fp32 result
    p.seg[g] = s;
    total += (long long)s.n_full * s.block_rows;
    p.row_end[g] = total;
  }
  p.n_segs = n_segs;
  p.d = d;
  p.n_subnets = n_subnets;
  p.live = n_subnets >= 32 ? live_subnets : (live_subnets & ((1u << n_subnets) - 1u));
  p.total_rows = total;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int grid = grid_for_rows(total);
  if (dtype == TWIST_BF16) aggregate_rows_kernel<true><<<grid, 256, 0, st>>>(p);
  else aggregate_rows_kernel<false><<<grid, 256, 0, st>>>(p);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}
