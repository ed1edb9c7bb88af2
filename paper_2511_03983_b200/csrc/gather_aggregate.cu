// twist_gather_subnets (dispatcher, Sec. 3.2) and twist_aggregate (aggregator, Sec. 3.3).
// Both are HBM-bandwidth kernels over whole rows (>= 1.5 KB in every workload, 8 KB at d_model = 4096
// in bf16).  The gather moves rows with the bulk-copy engine: global -> shared memory -> global, the
// fp32 master widened in shared memory on the way, so that the SMs issue almost no global-memory
// instructions.  The aggregate is one warp per row with 16-byte accesses per lane and several
// independent loads in flight.
#include "common.cuh"
#include "ptx.cuh"

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
  int parts;          // work item = one of `parts` equal spans of a row
  int part_chunks;    // float4 chunks per span
  int mode;           // AGG_MEAN: the aggregator; AGG_PARTIAL / AGG_FINISH: its two halves when the subnets are spread
                      // over several GPUs (sum over this GPU's subnets; division of the reduced sums by the coverage)
  int subnet_begin;   // AGG_PARTIAL: global index of this GPU's first subnet (bit of the cover masks)
};
enum { AGG_MEAN = 0, AGG_PARTIAL = 1, AGG_FINISH = 2 };

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
#ifndef TWIST_AGG_PART_CHUNKS
#define TWIST_AGG_PART_CHUNKS 256
#endif
constexpr int kAggPartChunks = TWIST_AGG_PART_CHUNKS;

#ifndef TWIST_GATHER_WARPS
#define TWIST_GATHER_WARPS 8
#define TWIST_GATHER_BUFS 2
#define TWIST_GATHER_AHEAD 1
#define TWIST_GATHER_PIECE 4096
#endif
constexpr int kGatherWarps = TWIST_GATHER_WARPS;        // warps per CTA
constexpr int kGatherBufs = TWIST_GATHER_BUFS;          // shared-memory buffers per warp
constexpr int kGatherAhead = TWIST_GATHER_AHEAD;        // a piece's load is requested this many items early
constexpr int kGatherPending = kGatherBufs - 1 - kGatherAhead;   // store groups that may still be reading shared memory
constexpr int kGatherPieceBytes = TWIST_GATHER_PIECE;   // a row travels in pieces of at most this many bytes
static_assert(kGatherAhead >= 1 && kGatherPending >= 0, "buffer ring too short for the lookahead");

// Work item = (destination row, piece of the row); one warp per item at a time, a ring of buffers per warp so
// the loads of the next items overlap the widening and the stores of the current one.
// Shared memory per warp and buffer: the piece as loaded [piece bytes] and, when masters are written,
// its fp32 widening [2 x piece bytes].  ELEM = 2 (bf16) or 4 (fp32) bytes.
template <int ELEM>
__global__ void __launch_bounds__(kGatherWarps * 32) gather_rows_kernel(const __grid_constant__ GatherParams p,
                                                                        int piece_bytes, int pieces, int buf_bytes,
                                                                        int* status) {
  extern __shared__ __align__(128) unsigned char gsm[];
  __shared__ __align__(8) unsigned long long bars[kGatherWarps][kGatherBufs];
  __shared__ int abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) abort_flag = 0;
  if (lane == 0) {
    for (int i = 0; i < kGatherBufs; ++i) mbar_init(smem_u32(&bars[warp][i]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  __syncthreads();
  const uint32_t wbase = smem_u32(gsm) + (uint32_t)warp * (uint32_t)kGatherBufs * (uint32_t)buf_bytes;
  const int row_bytes = p.d * ELEM;
  const long long items = p.total_rows * pieces;
  const long long wid0 = (long long)blockIdx.x * kGatherWarps + warp;
  const long long stride = (long long)gridDim.x * kGatherWarps;

  // Item `it` decoded.  The kept-block index is loaded here but only used when the item's copy is requested,
  // one iteration later, so that its latency (it is rarely cached) stays off the critical path.
  struct Item {
    const char* src_base;   // null: a padding row, written as zeros
    long long src_row;      // row of the source piece before the block index is applied
    int block_rows, idxv, n_blocks, off;
    char* dst; char* mst; int bytes;
  };
  // A kept-block id outside the source's block range: the row is neither read nor written, the status word says so.
  auto bad_index = [](const Item& o) { return o.src_base && (unsigned)o.idxv >= (unsigned)o.n_blocks; };
  auto decode = [&](long long it) {
    Item o;
    o.src_base = nullptr; o.src_row = 0; o.block_rows = 0; o.idxv = 0; o.n_blocks = 0; o.off = 0; o.dst = nullptr; o.mst = nullptr; o.bytes = 0;
    if (it >= items) return o;
    const long long r = it / pieces;
    const int pc = (int)(it - r * pieces);
    int g = 0;
    while (g + 1 < p.n_segs && r >= p.row_end[g]) ++g;
    const twist_gather_segment& sg = p.seg[g];
    const long long rl = r - (g ? p.row_end[g - 1] : 0);
    const int rows_per_subnet = sg.n_keep * sg.block_rows;
    const int s = (int)(rl / rows_per_subnet);
    const int rem = (int)(rl - (long long)s * rows_per_subnet);
    const int j = rem / sg.block_rows, i = rem - j * sg.block_rows;
    const bool valid = sg.count ? (j < sg.count[s]) : true;
    const long long dst_elem = (long long)s * sg.dst_subnet_stride + (sg.dst_row_offset + rem) * p.d;
    o.off = pc * piece_bytes;
    o.bytes = min(piece_bytes, row_bytes - o.off);
    o.dst = static_cast<char*>(sg.dst) + dst_elem * ELEM + o.off;
    o.mst = (ELEM == 2 && sg.dst_master) ? reinterpret_cast<char*>(sg.dst_master + dst_elem) + 2 * o.off : nullptr;
    if (valid) {
      o.src_base = static_cast<const char*>(sg.src);
      o.src_row = sg.src_row_offset + i;
      o.block_rows = sg.block_rows;
      o.n_blocks = sg.n_blocks;
      asm volatile("ld.global.nc.s32 %0, [%1];" : "=r"(o.idxv) : "l"(sg.idx + (long long)s * sg.idx_stride + j));
    }
    return o;
  };
  auto request = [&](const Item& o, int b) {          // lane 0
    if (!o.src_base || bad_index(o)) return;
    const uint32_t bar = smem_u32(&bars[warp][b]);
    const char* src = o.src_base + (o.src_row + (long long)o.idxv * o.block_rows) * row_bytes + o.off;
    mbar_expect_tx(bar, (uint32_t)o.bytes);
    bulk_load(wbase + (uint32_t)b * buf_bytes, src, (uint32_t)o.bytes, bar);
  };

  // Ring discipline: item n lives in buffer n % kGatherBufs and commits exactly one store group (an empty one for
  // a padding row), so "at most kGatherPending groups still reading" frees the buffer of item n + kGatherAhead.
  uint32_t phase = 0;                                  // bit b: parity of buffer b's barrier
  Item q[kGatherAhead + 1];                            // q[0] current, q[1..] requested, q[kGatherAhead] decoded only
#pragma unroll
  for (int i = 0; i <= kGatherAhead; ++i) q[i] = decode(wid0 + i * stride);
#pragma unroll
  for (int i = 0; i < kGatherAhead; ++i)
    if (lane == 0) request(q[i], i % kGatherBufs);
  int b = 0, b_req = kGatherAhead % kGatherBufs;
  for (long long it = wid0; it < items; it += stride) {
    const Item fresh = decode(it + (kGatherAhead + 1) * stride);   // its index load is in flight during this iteration
    if (lane == 0) {
      bulk_wait_read<kGatherPending>();                // the stores that read buffer b_req are done with it
      request(q[kGatherAhead], b_req);
    }
    const Item cur = q[0];
    const uint32_t in = wbase + (uint32_t)b * buf_bytes;
    if (bad_index(cur)) {                              // skipped: destination row left as it was
      if (lane == 0) note_status(status, (int)TWIST_ERR_BAD_INDEX);
    } else if (cur.src_base) {
      const uint32_t parity = (phase >> b) & 1u;
      // warp-uniform outcome: either every lane goes on or every lane leaves
      if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars[warp][b]), parity, &abort_flag, status))) break;
      phase ^= 1u << b;
      if (lane == 0) bulk_store(cur.dst, in, (uint32_t)cur.bytes);
      if (cur.mst) {                                   // exact widening bf16 -> fp32, staged in shared memory
        const uint32_t out = in + (uint32_t)piece_bytes;
        for (int c = lane; c < cur.bytes / 16; c += 32) {
          const uint4 v = lds128(in + 16u * c);
          sts128(out + 32u * c, widen_lo(v));
          sts128(out + 32u * c + 16u, widen_hi(v));
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) bulk_store(cur.mst, out, 2u * (uint32_t)cur.bytes);
      }
    } else {                                           // padding row: zeros, plain stores
      for (int c = lane; c < cur.bytes / 16; c += 32) {
        st_cs(reinterpret_cast<uint4*>(cur.dst) + c, make_uint4(0, 0, 0, 0));
        if (cur.mst) {
          st_cs(reinterpret_cast<uint4*>(cur.mst) + 2 * c, make_uint4(0, 0, 0, 0));
          st_cs(reinterpret_cast<uint4*>(cur.mst) + 2 * c + 1, make_uint4(0, 0, 0, 0));
        }
      }
    }
    if (lane == 0) bulk_commit();
    __syncwarp();
#pragma unroll
    for (int i = 0; i < kGatherAhead; ++i) q[i] = q[i + 1];
    q[kGatherAhead] = fresh;
    b = b + 1 == kGatherBufs ? 0 : b + 1;
    b_req = b_req + 1 == kGatherBufs ? 0 : b_req + 1;
  }
  if (lane == 0) bulk_wait_read<0>();
  __syncthreads();
  drain_after_abort(&abort_flag);     // a wait expired: a copy may still be in flight towards shared memory
}

__device__ inline uint32_t pack_bf16x2_rn(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// One warp per full-model row: 16-byte accesses per lane, several independent loads in flight; fp32 sum over the
// covering subnets in ascending order, correctly rounded quotient.  (A bulk-copy version of this kernel, like the
// gather's, measured slower: 2 KB pieces keep too few bytes in flight per SM.)
template <bool BF16>
__global__ void __launch_bounds__(256) aggregate_rows_kernel(const __grid_constant__ AggParams p, int* status) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  const int chunks = p.d / 4;                          // float4 chunks per row
  const long long items = p.total_rows * p.parts;
  for (long long it = warp0; it < items; it += nwarps) {
    const long long r = it / p.parts;
    const int c_begin = (int)(it - r * p.parts) * p.part_chunks;
    const int c_end = c_begin + p.part_chunks < chunks ? c_begin + p.part_chunks : chunks;
    int g = 0;
    while (g + 1 < p.n_segs && r >= p.row_end[g]) ++g;
    const twist_aggregate_segment& sg = p.seg[g];
    const long long rl = r - (g ? p.row_end[g - 1] : 0);
    const int b = (int)(rl / sg.block_rows), i = (int)(rl - (long long)b * sg.block_rows);
    const uint32_t held = sg.cover[b] & p.live;          // subnets (global numbering) that hold the block
    // the rows this warp adds up: every holder (AGG_MEAN), this GPU's holders (AGG_PARTIAL: bits subnet_begin ..
    // subnet_begin + n_subnets - 1, renumbered from 0 - sub and pos hold only those), or the one row of reduced
    // sums (AGG_FINISH)
    uint32_t m = held;
    if (p.mode == AGG_PARTIAL) m = (held >> p.subnet_begin) & (p.n_subnets >= 32 ? 0xFFFFFFFFu : ((1u << p.n_subnets) - 1u));
    if (p.mode != AGG_PARTIAL && held == 0) continue;    // held by no live subnet: untouched
    const int cnt = p.mode == AGG_FINISH ? 1 : __popc(m);
    // lane k holds the row pointer of the k-th covering subnet; bit 0 marks a row of the full-width matrix itself
    // (it may be the destination, so it is read with an ordinary load, not through the read-only path)
    unsigned long long mine = 0;
    const long long drow = sg.dst_row_offset + rl;
    bool bad = false;
    if (lane < cnt) {
      const int s = p.mode == AGG_FINISH ? -1 : __fns(m, 0, lane + 1);
      if (p.mode == AGG_FINISH || (sg.central && s == sg.central_subnet)) {   // a row in full-matrix geometry
        mine = reinterpret_cast<unsigned long long>(sg.central + drow * p.d) | 1ull;
      } else {
        const int rank = sg.pos[(long long)s * sg.n_full + b];
        bad = (unsigned)rank >= (unsigned)sg.n_keep;     // not a row of the subnet's slice
        const long long srow = sg.sub_row_offset + (long long)rank * sg.block_rows + i;
        mine = reinterpret_cast<unsigned long long>(sg.sub + (long long)s * sg.sub_subnet_stride + srow * p.d);
      }
    }
    if (__any_sync(0xffffffffu, bad)) {                  // row left as it was, the status word says so
      if (lane == 0) note_status(status, (int)TWIST_ERR_BAD_INDEX);
      continue;
    }
    // Quotient by the coverage count: reciprocal product corrected with the exact remainder, which gives
    // the correctly rounded quotient (the same bits as an IEEE division) at a fraction of its cost.
    // (AGG_PARTIAL divides by one - the sum itself; AGG_FINISH by the number of holders on all GPUs)
    const float denom = p.mode == AGG_PARTIAL ? 1.f : (float)__popc(held);
    const float rden = 1.0f / denom;
    auto quot = [&](float a) {
      const float q = a * rden;
      return fmaf(fmaf(-q, denom, a), rden, q);
    };
    // warp-uniform trip count (the shuffles below need every lane): lanes past the end of the span load nothing
    for (int cb = c_begin; cb < c_end; cb += 32 * kUnroll) {
      const int c0 = cb + lane;
      float4 acc[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int k = 0; k < cnt; ++k) {
        const unsigned long long bits = __shfl_sync(0xffffffffu, mine, k);
        const uint4* ptr = reinterpret_cast<const uint4*>(bits & ~1ull);
        const bool in_place = (bits & 1ull) != 0;        // warp-uniform
        uint4 raw[kUnroll];
        if (!in_place) {                                 // the loads of one source are issued together
#pragma unroll
          for (int u = 0; u < kUnroll; ++u)
            raw[u] = (c0 + 32 * u < c_end) ? ld_nc(ptr + c0 + 32 * u) : make_uint4(0, 0, 0, 0);
        } else {
#pragma unroll
          for (int u = 0; u < kUnroll; ++u)
            raw[u] = (c0 + 32 * u < c_end) ? *(ptr + c0 + 32 * u) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
          acc[u].x += __uint_as_float(raw[u].x);
          acc[u].y += __uint_as_float(raw[u].y);
          acc[u].z += __uint_as_float(raw[u].z);
          acc[u].w += __uint_as_float(raw[u].w);
        }
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int c = c0 + 32 * u;
        if (c < c_end) {
          float4 q = make_float4(quot(acc[u].x), quot(acc[u].y), quot(acc[u].z), quot(acc[u].w));
          uint4 qb = make_uint4(__float_as_uint(q.x), __float_as_uint(q.y), __float_as_uint(q.z), __float_as_uint(q.w));
          if (BF16) {
            if (sg.dst_f32) st_cs(reinterpret_cast<uint4*>(sg.dst_f32 + drow * p.d) + c, qb);
            if (p.mode != AGG_PARTIAL)                   // partial sums are fp32 only
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

int grid_for_items(long long items) {
  const long long warps_per_cta = 8;
  long long want = (items + warps_per_cta - 1) / warps_per_cta;
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
    if (s.n_keep <= 0 || s.block_rows <= 0 || s.n_blocks <= 0 || s.idx_stride < s.n_keep || s.src_row_offset < 0 ||
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
  bool any_master = false;
  for (int g = 0; g < n_segs; ++g) any_master |= segs[g].dst_master != nullptr;
  const int row_bytes = d * elem;
  const int piece_bytes = row_bytes < kGatherPieceBytes ? row_bytes : kGatherPieceBytes;
  const int pieces = (row_bytes + piece_bytes - 1) / piece_bytes;
  const int buf_bytes = piece_bytes * (any_master ? 3 : 1);          // the piece + its fp32 widening
  const int smem = kGatherWarps * kGatherBufs * buf_bytes;
  static bool configured[64] = {false};
  const int slot = device_slot();
  if (!configured[slot]) {
    TWIST_CUDA_TRY(cudaFuncSetAttribute(gather_rows_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        kGatherWarps * kGatherBufs * 3 * kGatherPieceBytes));
    TWIST_CUDA_TRY(cudaFuncSetAttribute(gather_rows_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        kGatherWarps * kGatherBufs * kGatherPieceBytes));
    configured[slot] = true;
  }
  // persistent grid: as many CTAs per SM as the shared memory allows (at most 8), or fewer for small inputs
  int per_sm = (220 * 1024) / (smem + 1024);
  per_sm = per_sm < 1 ? 1 : (per_sm > 8 ? 8 : per_sm);
  const long long items = total * pieces;
  const long long want = (items + kGatherWarps - 1) / kGatherWarps;
  const long long cap = (long long)sm_count() * per_sm;
  const int grid = (int)(want < cap ? (want > 0 ? want : 1) : cap);
  int* status = device_status_ptr();
  if (!status) return TWIST_ERR_CUDA;
  if (dtype == TWIST_BF16)
    gather_rows_kernel<2><<<grid, kGatherWarps * 32, smem, st>>>(p, piece_bytes, pieces, buf_bytes, status);
  else
    gather_rows_kernel<4><<<grid, kGatherWarps * 32, smem, st>>>(p, piece_bytes, pieces, buf_bytes, status);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

namespace twist {
namespace {
int aggregate_launch(const twist_aggregate_segment* segs, int n_segs, int n_subnets, int subnet_begin, int d, int dtype,
                     uint32_t live_subnets, int mode, void* stream) {
  if (!segs) return TWIST_ERR_NULL;
  if (n_segs <= 0 || n_segs > TWIST_MAX_SEGMENTS || n_subnets <= 0 || n_subnets > TWIST_MAX_SUBNETS || d <= 0)
    return TWIST_ERR_SHAPE;
  if (subnet_begin < 0 || subnet_begin + n_subnets > TWIST_MAX_SUBNETS) return TWIST_ERR_SHAPE;
  if (dtype != TWIST_FP32 && dtype != TWIST_BF16) return TWIST_ERR_SHAPE;
  if (d % 4 != 0 || (dtype == TWIST_BF16 && d % 8 != 0)) return TWIST_ERR_SHAPE;
  AggParams p;
  memset(&p, 0, sizeof(p));
  long long total = 0;
  for (int g = 0; g < n_segs; ++g) {
    const twist_aggregate_segment& s = segs[g];
    if (!s.dst || !s.cover) return TWIST_ERR_NULL;
    if (mode != AGG_FINISH && (!s.sub || !s.pos)) return TWIST_ERR_NULL;
    if (mode == AGG_FINISH && !s.central) return TWIST_ERR_NULL;                  // the reduced sums
    if (mode == AGG_PARTIAL && s.central) return TWIST_ERR_UNSUPPORTED;           // no in-place worker on a shard
    if (mode == AGG_PARTIAL && dtype == TWIST_BF16 && !s.dst_f32) return TWIST_ERR_NULL;   // sums are fp32
    if (s.n_full <= 0 || s.block_rows <= 0 || s.dst_row_offset < 0) return TWIST_ERR_SHAPE;
    if (mode != AGG_FINISH && (s.n_keep <= 0 || s.sub_row_offset < 0 || s.sub_subnet_stride < 0 || s.sub_subnet_stride % 4 != 0))
      return TWIST_ERR_SHAPE;
    if (!aligned16(s.dst) || !aligned16(s.sub) || !aligned16(s.dst_f32) || !aligned16(s.central)) return TWIST_ERR_SHAPE;
    if (mode == AGG_MEAN && s.central && (s.central_subnet < 0 || s.central_subnet >= n_subnets)) return TWIST_ERR_BAD_INDEX;
    if (dtype == TWIST_FP32 && s.dst_f32) return TWIST_ERR_UNSUPPORTED;      // dst already is the fp32 result
    p.seg[g] = s;
    total += (long long)s.n_full * s.block_rows;
    p.row_end[g] = total;
  }
  p.n_segs = n_segs;
  p.d = d;
  p.n_subnets = n_subnets;
  p.mode = mode;
  p.subnet_begin = subnet_begin;
  // cover masks number the subnets globally: AGG_MEAN and AGG_FINISH see n_subnets of them from bit 0, AGG_PARTIAL
  // keeps every live bit and picks its own range in the kernel
  p.live = (mode == AGG_PARTIAL || n_subnets >= 32) ? live_subnets : (live_subnets & ((1u << n_subnets) - 1u));
  p.total_rows = total;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // A row is split into spans of kAggPartChunks float4 chunks: with whole rows as items a warp of the persistent
  // grid gets only a handful, and the slowest warp (one row more, or rows with more covering subnets) sets the time.
  p.part_chunks = kAggPartChunks;
  p.parts = (d / 4 + kAggPartChunks - 1) / kAggPartChunks;
  const int grid = grid_for_items(total * p.parts);
  int* status = device_status_ptr();
  if (!status) return TWIST_ERR_CUDA;
  if (dtype == TWIST_BF16) aggregate_rows_kernel<true><<<grid, 256, 0, st>>>(p, status);
  else aggregate_rows_kernel<false><<<grid, 256, 0, st>>>(p, status);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}
}  // namespace
}  // namespace twist

extern "C" int32_t twist_aggregate(const twist_aggregate_segment* segs, int32_t n_segs, int32_t n_subnets, int32_t d,
                                   int32_t dtype, uint32_t live_subnets, void* stream) {
  return twist::aggregate_launch(segs, n_segs, n_subnets, 0, d, dtype, live_subnets, twist::AGG_MEAN, stream);
}

extern "C" int32_t twist_aggregate_partial(const twist_aggregate_segment* segs, int32_t n_segs, int32_t n_subnets,
                                           int32_t subnet_begin, int32_t d, int32_t dtype, uint32_t live_subnets,
                                           void* stream) {
  return twist::aggregate_launch(segs, n_segs, n_subnets, subnet_begin, d, dtype, live_subnets, twist::AGG_PARTIAL, stream);
}

extern "C" int32_t twist_aggregate_finish(const twist_aggregate_segment* segs, int32_t n_segs, int32_t n_subnets, int32_t d,
                                          int32_t dtype, uint32_t live_subnets, void* stream) {
  return twist::aggregate_launch(segs, n_segs, n_subnets, 0, d, dtype, live_subnets, twist::AGG_FINISH, stream);
}
