// Routing decision + query compaction (Eq. 3; Section 3.2; Algorithm 1 step 1), and the row gather
// that consolidates routed rows into a contiguous buffer.
//
// Two small launches, both HBM/latency bound:
//   route_count : each CTA thresholds 4096 positions and counts its routed ones (ballot + popc)
//   route_scan  : each CTA sums the counts of the CTAs before it, rescans its own 4096 positions
//                 (per-thread popcount of a 16-bit flag word, warp shuffle scan, cross-warp scan)
//                 and writes d_mask, prefix, q_idx (ascending = stable) and the -1 tail.
// Nothing is read back by the host: the routed count stays on the device.
#include "l2a_common.cuh"

namespace l2a {

namespace {

constexpr int kThreads = 256;
constexpr int kPerThread = kRouteBlockElems / kThreads;  // 16

__device__ __forceinline__ uint32_t load_flags(const void* router, int kind, float thr, int64_t row_base, int t0,
                                               int L) {
  uint32_t flags = 0;
  if (kind == L2A_ROUTER_MASK_U8) {
    const uint8_t* m = static_cast<const uint8_t*>(router) + row_base;
    if (t0 + kPerThread <= L && ((reinterpret_cast<uintptr_t>(m + t0) & 15) == 0)) {
      const uint4 v = *reinterpret_cast<const uint4*>(m + t0);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if ((w[i] >> (8 * k)) & 0xffu) flags |= 1u << (4 * i + k);
    } else {
      for (int i = 0; i < kPerThread; ++i)
        if (t0 + i < L && m[t0 + i]) flags |= 1u << i;
    }
  } else if (kind == L2A_ROUTER_LOGITS_BF16) {
    const bf16* z = static_cast<const bf16*>(router) + row_base;
    for (int i = 0; i < kPerThread; ++i)
      if (t0 + i < L && __bfloat162float(z[t0 + i]) >= thr) flags |= 1u << i;   // the upcast is exact
  } else {
    const float* z = static_cast<const float*>(router) + row_base;
    for (int i = 0; i < kPerThread; ++i)
      if (t0 + i < L && z[t0 + i] >= thr) flags |= 1u << i;  // NaN compares false; -0.0 >= 0.0 is true
  }
  return flags;
}

__global__ void __launch_bounds__(kThreads) route_count_kernel(RouteArgs a) {
  const int b = blockIdx.y, blk = blockIdx.x;
  const int t0 = blk * kRouteBlockElems + threadIdx.x * kPerThread;
  const uint32_t flags = load_flags(a.router, a.router_kind, a.threshold, (int64_t)b * a.L, t0, a.L);
  int cnt = __popc(flags);
  __shared__ int warp_cnt[kThreads / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
  if ((threadIdx.x & 31) == 0) warp_cnt[threadIdx.x >> 5] = cnt;
  __syncthreads();
  if (threadIdx.x == 0) {
    int s = 0;
    for (int w = 0; w < kThreads / 32; ++w) s += warp_cnt[w];
    a.block_sums[b * a.nblocks + blk] = s;
  }
}

__global__ void __launch_bounds__(kThreads) route_scan_kernel(RouteArgs a) {
  const int b = blockIdx.y, blk = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __shared__ int red_before[kThreads / 32], red_total[kThreads / 32], warp_off[kThreads / 32];

  // counts of the CTAs before this one, and the row total
  int before = 0, total = 0;
  for (int i = threadIdx.x; i < a.nblocks; i += kThreads) {
    const int v = a.block_sums[b * a.nblocks + i];
    total += v;
    if (i < blk) before += v;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    before += __shfl_xor_sync(0xffffffffu, before, o);
    total += __shfl_xor_sync(0xffffffffu, total, o);
  }
  if (lane == 0) { red_before[warp] = before; red_total[warp] = total; }
  __syncthreads();
  before = 0; total = 0;
  for (int w = 0; w < kThreads / 32; ++w) { before += red_before[w]; total += red_total[w]; }

  const int t0 = blk * kRouteBlockElems + threadIdx.x * kPerThread;
  const uint32_t flags = load_flags(a.router, a.router_kind, a.threshold, (int64_t)b * a.L, t0, a.L);
  const int cnt = __popc(flags);
  int incl = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) warp_off[warp] = incl;
  __syncthreads();
  int c = before + incl - cnt;
  for (int w = 0; w < warp; ++w) c += warp_off[w];

  uint8_t* dm = a.d_mask + (int64_t)b * a.L;
  int32_t* qi = a.q_idx + (int64_t)b * a.L;
  int32_t* pf = a.prefix + (int64_t)b * (a.L + 1);
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    const int t = t0 + i;
    if (t < a.L) {
      const int on = (flags >> i) & 1;
      dm[t] = (uint8_t)on;
      pf[t] = c;
      if (on) qi[c++] = t;
      if (t >= total) qi[t] = -1;  // compact slots past the routed count
    }
  }
  if (blk == 0 && threadIdx.x == 0) {
    a.n_routed[b] = total;
    pf[a.L] = total;
  }
}

// One CTA per compact row (grid-stride); 16-byte chunks.
__global__ void __launch_bounds__(256) gather_rows_kernel(const bf16* __restrict__ src, bf16* __restrict__ dst,
                                                          const int32_t* __restrict__ q_idx,
                                                          const int32_t* __restrict__ n_routed, int L,
                                                          int row_chunks /* 16-byte chunks per row */,
                                                          const int32_t* __restrict__ prefix, int row_begin,
                                                          int row_end, int64_t src_batch_chunks,
                                                          int64_t src_row_chunks, int* status) {
  const int b = blockIdx.y;
  const int n_c = n_routed[b];
  int n_pad = (n_c + kRowsPerCta - 1) / kRowsPerCta * kRowsPerCta;
  if (n_pad > L) n_pad = L;
  // optional restriction to the routed rows t in [row_begin, row_end): they are the compact rows
  // [prefix[row_begin], prefix[row_end]); the zero padding belongs to the range that ends at L
  int c_begin = 0;
  if (prefix != nullptr) {
    c_begin = prefix[(int64_t)b * (L + 1) + row_begin];
    if (row_end < L) n_pad = prefix[(int64_t)b * (L + 1) + row_end];
  }
  const uint4* s = reinterpret_cast<const uint4*>(src) + b * src_batch_chunks;   // source strides in 16-byte chunks
  uint4* d = reinterpret_cast<uint4*>(dst) + (int64_t)b * L * row_chunks;
  for (int c = c_begin + blockIdx.x; c < n_pad; c += gridDim.x) {
    if (c < n_c) {
      const int t = q_idx[(int64_t)b * L + c];
      if (!dbg_in_range(t >= 0 && t < L, status)) continue;
      for (int i = threadIdx.x; i < row_chunks; i += blockDim.x)
        d[(int64_t)c * row_chunks + i] = __ldg(&s[t * src_row_chunks + i]);
    } else {
      for (int i = threadIdx.x; i < row_chunks; i += blockDim.x)
        d[(int64_t)c * row_chunks + i] = make_uint4(0, 0, 0, 0);
    }
  }
}

// Router logit (Eq. 3).  The grid is sized to the machine: the warps take groups of four tokens round-robin (the
// whole grid reads one contiguous stretch of S at a time), four at a time so that each 32-byte piece of w fetched
// (from L1) serves four 16-byte loads of S and several rows are in flight per warp; fp32 accumulation.
constexpr int kRlTokens = 4;
__global__ void __launch_bounds__(256) router_logits_kernel(const bf16* __restrict__ S, const float* __restrict__ w,
                                                            float bias, float* __restrict__ logits,
                                                            float* __restrict__ sum_sq, int B, int L, int row_elems) {
  const int64_t n_tokens = (int64_t)B * L;
  const int64_t n_warps = (int64_t)gridDim.x * (blockDim.x >> 5);
  const int64_t gw = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int64_t t_begin = gw * kRlTokens, t_end = n_tokens;
  const int n_chunks = row_elems / 8;
  const float4* w4 = reinterpret_cast<const float4*>(w);
  // sum of sigmoid^2 of this warp's tokens, flushed with one atomic per batch entry they touch (the batch index
  // never decreases along a warp's tokens)
  float reg_sum = 0.f;
  int64_t reg_b = t_begin < t_end ? t_begin / L : 0;
  for (int64_t token0 = t_begin; token0 < t_end; token0 += n_warps * kRlTokens) {
    const uint4* rows[kRlTokens];
    float acc[kRlTokens];
#pragma unroll
    for (int r = 0; r < kRlTokens; ++r) {
      // rows past the range re-read its last token; their result is not stored
      const int64_t tok = token0 + r < t_end ? token0 + r : t_end - 1;
      rows[r] = reinterpret_cast<const uint4*>(S) + tok * n_chunks;
      acc[r] = 0.f;
    }
#pragma unroll 2
    for (int i = lane; i < n_chunks; i += 32) {
      uint4 v[kRlTokens];
#pragma unroll
      for (int r = 0; r < kRlTokens; ++r) v[r] = __ldg(&rows[r][i]);
      const float4 wa = __ldg(&w4[2 * i]), wb = __ldg(&w4[2 * i + 1]);
      const float ww[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
#pragma unroll
      for (int r = 0; r < kRlTokens; ++r) {
        const uint32_t u[4] = {v[r].x, v[r].y, v[r].z, v[r].w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          acc[r] = fmaf(__uint_as_float(u[k] << 16), ww[2 * k], acc[r]);
          acc[r] = fmaf(__uint_as_float(u[k] & 0xffff0000u), ww[2 * k + 1], acc[r]);
        }
      }
    }
#pragma unroll
    for (int r = 0; r < kRlTokens; ++r) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc[r] += __shfl_xor_sync(0xffffffffu, acc[r], o);
      if (lane == 0 && token0 + r < t_end) {
        const float z = acc[r] + bias;
        logits[token0 + r] = z;
        if (sum_sq != nullptr) {
          const float g = 1.0f / (1.0f + __expf(-z));
          const int64_t bb = (token0 + r) / L;
          if (bb != reg_b) {
            atomicAdd(&sum_sq[reg_b], reg_sum);
            reg_sum = 0.f;
            reg_b = bb;
          }
          reg_sum += g * g;
        }
      }
    }
  }
  if (sum_sq != nullptr && lane == 0 && t_end > t_begin) atomicAdd(&sum_sq[reg_b], reg_sum);
}

// Packed variable-length batches: token t belongs to the sequence i with cu[i] <= t < cu[i + 1] (binary search over
// the n_seq + 1 boundaries); tokens at or after cu[n_seq] are sequences of their own.
__global__ void __launch_bounds__(256) pack_sequences_kernel(const int32_t* __restrict__ cu, int n_seq, int L,
                                                             int32_t* __restrict__ seq_bounds) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= L) return;
  int lo = 0, hi = n_seq;                  // invariant: cu[lo] <= t (cu[0] = 0); answer in [lo, hi)
  if (n_seq <= 0 || t >= __ldg(&cu[n_seq])) {
    reinterpret_cast<int2*>(seq_bounds)[t] = make_int2(t, t + 1);
    return;
  }
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (__ldg(&cu[mid]) <= t) lo = mid; else hi = mid;
  }
  int first = __ldg(&cu[lo]), end = __ldg(&cu[lo + 1]);
  // boundaries that are not ascending must still give a range that holds t and stays inside the axis
  first = max(0, min(first, t));
  end = min(L, max(end, t + 1));
  reinterpret_cast<int2*>(seq_bounds)[t] = make_int2(first, end);
}

}  // namespace

cudaError_t launch_router_logits(const bf16* S, const float* w, float bias, float* logits, float* sum_sq, int B, int L,
                                 int row_elems, cudaStream_t stream) {
  int device = 0, sms = 148;
  if (cudaGetDevice(&device) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
  int per_sm = 0;   // one resident wave: every CTA of the grid runs at once and owns an equal share
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, router_logits_kernel, 256, 0) != cudaSuccess || per_sm < 1)
    per_sm = 1;
  int64_t blocks = (int64_t)sms * per_sm;
  const int64_t max_blocks = ((int64_t)B * L + 8 * kRlTokens - 1) / (8 * kRlTokens);
  if (blocks > max_blocks) blocks = max_blocks;
  router_logits_kernel<<<(unsigned)blocks, 256, 0, stream>>>(S, w, bias, logits, sum_sq, B, L, row_elems);
  return cudaGetLastError();
}

cudaError_t launch_pack_sequences(const int32_t* cu_seqlens, int n_seq, int L, int32_t* seq_bounds, cudaStream_t stream) {
  pack_sequences_kernel<<<ceil_div(L, 256), 256, 0, stream>>>(cu_seqlens, n_seq, L, seq_bounds);
  return cudaGetLastError();
}

cudaError_t launch_route_compact(const RouteArgs& a, cudaStream_t stream) {
  dim3 grid(a.nblocks, a.B);
  route_count_kernel<<<grid, kThreads, 0, stream>>>(a);
  route_scan_kernel<<<grid, kThreads, 0, stream>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_gather_rows(const bf16* src, bf16* dst, const int32_t* q_idx, const int32_t* n_routed, int B,
                               int L, int row_elems, cudaStream_t stream, const int32_t* prefix, int row_begin,
                               int row_end, RowStrides src_strides, int* status) {
  const int row_chunks = row_elems * 2 / 16;
  const int64_t ts = src_strides.t > 0 ? src_strides.t : row_elems;
  const int64_t bs = src_strides.b > 0 ? src_strides.b : (int64_t)L * ts;
  int gx = L < 148 * 16 ? L : 148 * 16;
  dim3 grid(gx, B);
  gather_rows_kernel<<<grid, 256, 0, stream>>>(src, dst, q_idx, n_routed, L, row_chunks, prefix, row_begin, row_end,
                                               bs / 8, ts / 8, status);
  return cudaGetLastError();
}

}  // namespace l2a

// ------------------------------------------------------------------------------------------------
// Variant of the routing/compaction entry point that needs no scratch from the caller and allocates
// nothing: the per-CTA counts live in a fixed array in the library's own device image.
//
// In host code `g_static_route_counts` is only a handle for the runtime, not a device address, so
// the launcher is never given the symbol itself: the address is looked up once per device with
// cudaGetSymbolAddress (with that device current) and cached.
static __device__ __align__(256) int32_t g_static_route_counts[L2A_STATIC_ROUTE_SLOTS];

namespace {
constexpr int kMaxDevices = 64;
int32_t* g_static_counts_addr[kMaxDevices] = {};

// Returns the device address of the static array on the current device (nullptr on failure).
int32_t* static_counts_for_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  int32_t* cached = __atomic_load_n(&g_static_counts_addr[dev], __ATOMIC_ACQUIRE);
  if (cached) return cached;
  void* ptr = nullptr;
  if (cudaGetSymbolAddress(&ptr, g_static_route_counts) != cudaSuccess || ptr == nullptr) return nullptr;
  __atomic_store_n(&g_static_counts_addr[dev], static_cast<int32_t*>(ptr), __ATOMIC_RELEASE);
  return static_cast<int32_t*>(ptr);
}
}  // namespace

extern "C" l2a_status l2a_route_compact_static(const l2a_params* p, const void* router, int router_kind,
                                               float logit_threshold, uint8_t* d_mask, int32_t* q_idx,
                                               int32_t* n_routed, int32_t* prefix, void* stream) {
  // shape checks come from the workspace query (host only, launches nothing)
  size_t unused = 0;
  l2a_status st = l2a_workspace_bytes(p, &unused, nullptr, nullptr);
  if (st != L2A_OK) return st;
  if (!router || !d_mask || !q_idx || !n_routed || !prefix) return L2A_ERR_INVALID_ARG;
  if (router_kind != L2A_ROUTER_MASK_U8 && router_kind != L2A_ROUTER_LOGITS_F32 &&
      router_kind != L2A_ROUTER_LOGITS_BF16)
    return L2A_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q_idx) | reinterpret_cast<uintptr_t>(n_routed) |
       reinterpret_cast<uintptr_t>(prefix)) & 3)
    return L2A_ERR_INVALID_ARG;
  if (router_kind == L2A_ROUTER_LOGITS_F32 && (reinterpret_cast<uintptr_t>(router) & 3)) return L2A_ERR_INVALID_ARG;
  if (router_kind == L2A_ROUTER_LOGITS_BF16 && (reinterpret_cast<uintptr_t>(router) & 1)) return L2A_ERR_INVALID_ARG;
  const int nblocks = l2a::ceil_div(p->Lq, l2a::kRouteBlockElems);
  if ((int64_t)p->B * nblocks > L2A_STATIC_ROUTE_SLOTS) return L2A_ERR_UNSUPPORTED;  // beyond the fixed scratch
  int32_t* counts = static_counts_for_current_device();
  if (!counts) return L2A_ERR_CUDA;
  l2a::RouteArgs a;
  a.router = router;
  a.router_kind = router_kind;
  a.threshold = logit_threshold;
  a.B = p->B;
  a.L = p->Lq;
  a.d_mask = d_mask;
  a.q_idx = q_idx;
  a.n_routed = n_routed;
  a.prefix = prefix;
  a.block_sums = counts;
  a.nblocks = nblocks;
  return l2a::launch_route_compact(a, static_cast<cudaStream_t>(stream)) == cudaSuccess ? L2A_OK : L2A_ERR_CUDA;
}
