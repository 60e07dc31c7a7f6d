// Decode step of the layer (Section 3.4): one new query token per sequence attends to the last W+1 keys of the
// cache (Local Attention) and, only if its routing decision d = 1, to the whole cache (Global Attention);
// o = s + d * a.  The work is one pass over the K/V cache: HBM-bound.  The cache of every KV head is split into
// chunks processed by independent CTAs (partial soft-max per chunk), merged by a second small kernel.
//
// Split kernel, one CTA = one chunk of keys of one (batch entry, KV head), for all G query heads of the group:
//   producer warp : streams 64-key K and V tiles through a ring of shared-memory stages with TMA (one 4-D copy
//                   per tile, 128-byte swizzle), so tens of KB per SM are in flight whatever the compute warps do.
//   compute warps : each takes 16 keys of every stage.  The G query heads are the rows of a 16-row MMA A operand
//                   (mma.sync m16n8k16, bf16 in, fp32 accumulate): S = Q K^T from ldmatrix'd K rows, running
//                   soft-max in the exp2 domain on the accumulator fragment, O += P V from transposed ldmatrix of
//                   the V rows.  The tensor cores are used only to keep the instruction count per key low enough
//                   that the copy engine, not instruction issue, sets the pace.
#include <math.h>

#include "l2a_common.cuh"
#include "sm100_prims.cuh"

namespace l2a {

namespace {

constexpr int kDecKeys = 64;                 // keys per pipeline stage
constexpr int kDecStages = 3;
constexpr int kDecComputeWarps = kDecKeys / 16;
constexpr int kDecThreads = (kDecComputeWarps + 1) * 32;   // + the producer warp
constexpr int kMaxGroup = 8;                 // query heads per KV head supported (rows 0..7 of the A operand)

struct DecodeArgs {
  int B, Lk, Hq, Hkv, G;
  int window, q_pos;       // the new token sits at position q_pos (normally Lk - 1)
  float scale_log2;
  int n_loc, n_glb;        // chunks of the local / global key range
  const bf16* q;           // [B, Hq, D]
  const uint8_t* d;        // [B] routing decision of the new token (NULL = never routed)
  float* part;             // [B, Hq, n_loc + n_glb, D + 2]  (acc[D], m, l)
  bf16* O;                 // [B, Hq, D]
  int* status;             // workspace status word
};

struct DecodeBars {
  uint64_t full[kDecStages], empty[kDecStages];
  int abort_flag;
};

template <int D>
constexpr size_t decode_smem_bytes() {
  return (size_t)kDecStages * 2 * kDecKeys * D * 2 + sizeof(DecodeBars);
}

__device__ __forceinline__ void chunk_range(int lo, int hi, int n, int i, int& c_lo, int& c_hi) {
  const int len = hi - lo + 1;
  int per = (len + n - 1) / n;
  per = (per + kDecKeys - 1) / kDecKeys * kDecKeys;
  c_lo = lo + i * per;
  c_hi = min(hi, c_lo + per - 1);
}

__device__ __forceinline__ void ldsm_x4(uint32_t saddr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(saddr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t saddr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(saddr));
}
// D += A * B, A 16x16 (row), B 16x8 (col), bf16 operands, fp32 accumulators.  Rows 8..15 of A are zero here.
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

// Address of the 16-byte chunk `chunk` (8 columns) of key row `row` inside a 64-key tile stored as D/64
// consecutive 128-byte-swizzled sub-tiles of 64 rows x 64 columns.
__device__ __forceinline__ uint32_t tile_addr(uint32_t tile, int row, int chunk) {
  return tile + (chunk >> 3) * (kDecKeys * 128) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4);
}

template <int D, int G>
__global__ void __launch_bounds__(kDecThreads, 2)
decode_split_kernel(const DecodeArgs a, const __grid_constant__ CUtensorMap mapK,
                    const __grid_constant__ CUtensorMap mapV) {
  constexpr int kTileBytes = kDecKeys * D * 2;
  constexpr int kStageBytes = 2 * kTileBytes;       // K tile, then V tile
  const int item = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const bool glb = item >= a.n_loc;
  if (glb && (a.d == nullptr || a.d[b] == 0)) return;          // Global Attention is skipped when d = 0
  const int lo = glb ? 0 : max(0, a.q_pos - a.window);
  int c_lo, c_hi;
  chunk_range(lo, a.q_pos, glb ? a.n_glb : a.n_loc, glb ? item - a.n_loc : item, c_lo, c_hi);
  const int n_tiles = c_hi >= c_lo ? (c_hi - c_lo) / kDecKeys + 1 : 0;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  extern __shared__ __align__(1024) uint8_t smem[];
  DecodeBars* bar = reinterpret_cast<DecodeBars*>(smem + kDecStages * kStageBytes);
  volatile int* abort_flag = &bar->abort_flag;
  if ((smem_u32(smem) & 1023u) != 0) {       // the swizzled tile addressing needs a 1024-byte-aligned base
    if (tid == 0) atomicExch(a.status, 2);
    return;
  }
  if (tid == 0) {
    for (int s = 0; s < kDecStages; ++s) {
      mbar_init(&bar->full[s], 1);
      mbar_init(&bar->empty[s], kDecComputeWarps);
    }
    bar->abort_flag = 0;
    fence_mbar_init();
  }
  __syncthreads();

  // per-thread soft-max state of head `hr` (accumulator row) over this warp's keys
  const int hr = lane >> 2, t4 = lane & 3;
  float m_run = -INFINITY, l_run = 0.f;
  float acc[D / 8][4];
#pragma unroll
  for (int j = 0; j < D / 8; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;

  if (warp == kDecComputeWarps) {
    // ================================================================= producer
    if (lane == 0) {
      tma_prefetch_desc(&mapK);
      tma_prefetch_desc(&mapV);
      for (int i = 0; i < n_tiles; ++i) {
        const int s = i % kDecStages, ph = (i / kDecStages) & 1;
        if (!mbar_wait(&bar->empty[s], ph ^ 1, abort_flag)) break;
        uint8_t* stage = smem + s * kStageBytes;
        mbar_expect_tx(&bar->full[s], kStageBytes);
        tma_load_4d(stage, &mapK, &bar->full[s], 0, c_lo + i * kDecKeys, g * (D / 64), b);
        tma_load_4d(stage + kTileBytes, &mapV, &bar->full[s], 0, c_lo + i * kDecKeys, g * (D / 64), b);
      }
    }
  } else {
    // ================================================================= compute warps
    // A fragments of Q: row hr = query head g*G + hr (zero rows for hr >= G), all D columns
    uint32_t qa[D / 16][2];
    {
      const bf16* qrow = a.q + ((int64_t)b * a.Hq + g * G + (hr < G ? hr : 0)) * D;
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        const uint32_t v0 = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * t4);
        const uint32_t v1 = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8 + 2 * t4);
        qa[ks][0] = hr < G ? v0 : 0u;
        qa[ks][1] = hr < G ? v1 : 0u;
      }
    }
    const int r0 = warp * 16;                          // this warp's key rows inside a stage
    const int lm = lane >> 3, lr = lane & 7;           // ldmatrix: lane -> (matrix, row of the matrix)
    const int k_row = r0 + (lm >> 1) * 8 + lr;         // K: matrices (keys lo|d lo), (keys lo|d hi), (keys hi|..)
    const int v_row = r0 + (lm & 1) * 8 + lr;          // V: matrices (keys lo|cols j), (keys hi|cols j), (..|j+1)

    for (int i = 0; i < n_tiles; ++i) {
      const int s = i % kDecStages, ph = (i / kDecStages) & 1;
      if (!mbar_wait_warp(&bar->full[s], ph, abort_flag)) break;
      const uint32_t tK = smem_u32(smem + s * kStageBytes), tV = tK + kTileBytes;
      const int key0 = c_lo + i * kDecKeys + r0;       // first key of this warp's 16
      if (key0 <= c_hi) {
        const bool tail = key0 + 15 > c_hi;
        // ---- S = Q K^T for 16 keys (two 8-key accumulator tiles)
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          uint32_t kb[4];
          ldsm_x4(tile_addr(tK, k_row, ks * 2 + (lm & 1)), kb);
          mma_16816(s0, qa[ks][0], qa[ks][1], kb[0], kb[1]);
          mma_16816(s1, qa[ks][0], qa[ks][1], kb[2], kb[3]);
        }
        // this thread: head hr, keys key0 + 2*t4 + {0, 1} (s0) and key0 + 8 + 2*t4 + {0, 1} (s1)
        float sc[4] = {s0[0] * a.scale_log2, s0[1] * a.scale_log2, s1[0] * a.scale_log2, s1[1] * a.scale_log2};
        uint32_t vm0 = 0xffffffffu, vm1 = 0xffffffffu;
        if (tail) {
          const int kq = key0 + 2 * t4;
          if (kq > c_hi) { sc[0] = -INFINITY; vm0 &= 0xffff0000u; }
          if (kq + 1 > c_hi) { sc[1] = -INFINITY; vm0 &= 0x0000ffffu; }
          if (kq + 8 > c_hi) { sc[2] = -INFINITY; vm1 &= 0xffff0000u; }
          if (kq + 9 > c_hi) { sc[3] = -INFINITY; vm1 &= 0x0000ffffu; }
        }
        float mx = fmaxf(fmaxf(sc[0], sc[1]), fmaxf(sc[2], sc[3]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run, mx);          // finite: key0 <= c_hi, so key 0 of the 16 is valid
        const float alpha = exp2f(m_run - m_new);      // 0 on the first step (m_run = -inf)
        const float p0 = exp2f(sc[0] - m_new), p1 = exp2f(sc[1] - m_new);
        const float p2 = exp2f(sc[2] - m_new), p3 = exp2f(sc[3] - m_new);
        l_run = l_run * alpha + ((p0 + p1) + (p2 + p3));   // per-thread partial sum, reduced at the end
        m_run = m_new;
        if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
          for (int j = 0; j < D / 8; ++j) { acc[j][0] *= alpha; acc[j][1] *= alpha; }
        }
        const uint32_t pa0 = pack_bf16(p0, p1), pa2 = pack_bf16(p2, p3);
        // ---- O += P V: B fragments are the transposed 8x8 blocks of the V rows
#pragma unroll
        for (int jj = 0; jj < D / 16; ++jj) {
          uint32_t vb[4];
          ldsm_x4_t(tile_addr(tV, v_row, jj * 2 + (lm >> 1)), vb);
          if (tail) { vb[0] &= vm0; vb[1] &= vm1; vb[2] &= vm0; vb[3] &= vm1; }   // rows past the chunk may hold anything
          mma_16816(acc[2 * jj], pa0, pa2, vb[0], vb[1]);
          mma_16816(acc[2 * jj + 1], pa0, pa2, vb[2], vb[3]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar->empty[s]);
    }
  }

  // ---- merge the compute warps of this CTA (stage memory is free once every warp has left the loop), then
  // write the chunk's partial result
  __syncthreads();
  float* red_acc = reinterpret_cast<float*>(smem);                           // [warps][G][D]
  float* red_m = red_acc + kDecComputeWarps * G * D;                         // [warps][G]
  float* red_l = red_m + kDecComputeWarps * G;
  float ls = l_run;
  ls += __shfl_xor_sync(0xffffffffu, ls, 1);
  ls += __shfl_xor_sync(0xffffffffu, ls, 2);
  if (warp < kDecComputeWarps && hr < G) {
    if (t4 == 0) { red_m[warp * G + hr] = m_run; red_l[warp * G + hr] = ls; }
#pragma unroll
    for (int j = 0; j < D / 8; ++j)
      *reinterpret_cast<float2*>(&red_acc[(warp * G + hr) * D + j * 8 + 2 * t4]) = make_float2(acc[j][0], acc[j][1]);
  }
  __syncthreads();
  const int n_items = a.n_loc + a.n_glb;
  for (int i = tid; i < G * D; i += kDecThreads) {
    const int h = i / D, col = i % D;
    float M = -INFINITY;
    for (int w = 0; w < kDecComputeWarps; ++w) M = fmaxf(M, red_m[w * G + h]);
    float L = 0.f, A = 0.f;
    for (int w = 0; w < kDecComputeWarps; ++w) {
      const float mw = red_m[w * G + h];
      const float f = (mw == -INFINITY) ? 0.f : exp2f(mw - M);
      L += red_l[w * G + h] * f;
      A += red_acc[(w * G + h) * D + col] * f;
    }
    float* dst = a.part + (((int64_t)b * a.Hq + g * G + h) * n_items + item) * (D + 2);
    dst[col] = A;
    if (col == 0) { dst[D] = M; dst[D + 1] = L; }
  }
  if (bar->abort_flag) {
    // a bounded wait ran out: give copies still in flight time to land before shared memory is released
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    if (tid == 0) atomicExch(a.status, 1);
    __syncthreads();
  }
}

// Merges the chunk partials of one (batch entry, query head): s over the local chunks, a over the global ones.
template <int D>
__global__ void __launch_bounds__(D) decode_merge_kernel(const DecodeArgs a) {
  const int h = blockIdx.x, b = blockIdx.y, col = threadIdx.x;
  const int n_items = a.n_loc + a.n_glb;
  const float* base = a.part + (((int64_t)b * a.Hq + h) * n_items) * (D + 2);
  const bool routed = a.d != nullptr && a.d[b] != 0;
  float out = 0.f;
  for (int pass = 0; pass < (routed ? 2 : 1); ++pass) {
    const int i0 = pass == 0 ? 0 : a.n_loc, i1 = pass == 0 ? a.n_loc : n_items;
    float M = -INFINITY;
    for (int i = i0; i < i1; ++i) M = fmaxf(M, base[i * (D + 2) + D]);
    float L = 0.f, A = 0.f;
    for (int i = i0; i < i1; ++i) {
      const float mi = base[i * (D + 2) + D];
      const float f = (mi == -INFINITY) ? 0.f : exp2f(mi - M);
      L += base[i * (D + 2) + D + 1] * f;
      A += base[i * (D + 2) + col] * f;
    }
    out += A / L;
  }
  a.O[((int64_t)b * a.Hq + h) * D + col] = __float2bfloat16(out);
}

void plan_chunks(const l2a_params* p, int* n_loc, int* n_glb) {
  // Cache chunks of at most 2048 keys, shrunk (down to 512) when few (sequence, KV head) pairs exist so that the
  // grid still covers the SMs a few times over; CTAs of non-routed sequences exit at once.  Local chunks of 256
  // keys.  The merge reads at most 512 + 64 partials per head.
  const int pos = p->q_pos_offset;
  const int local_len = (pos < p->window ? pos : p->window) + 1;
  const int64_t pairs = (int64_t)p->B * p->Hkv;
  int64_t per = ((int64_t)(pos + 1) * pairs + 1183) / 1184;
  per = per < 512 ? 512 : (per > 2048 ? 2048 : per);
  int ng = ceil_div(pos + 1, (int)per);
  if (ng > 512) ng = 512;
  int nl = ceil_div(local_len, 256);
  if (nl > 64) nl = 64;
  *n_loc = nl < 1 ? 1 : nl;
  *n_glb = ng < 1 ? 1 : ng;
}

template <int D, int G>
cudaError_t launch_split(const DecodeArgs& a, const CUtensorMap& mapK, const CUtensorMap& mapV, dim3 grid,
                         cudaStream_t s) {
  constexpr size_t smem = decode_smem_bytes<D>();
  cudaError_t e = cudaFuncSetAttribute(decode_split_kernel<D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  decode_split_kernel<D, G><<<grid, kDecThreads, smem, s>>>(a, mapK, mapV);
  return cudaGetLastError();
}

template <int D>
cudaError_t launch_split_d(const DecodeArgs& a, const CUtensorMap& mapK, const CUtensorMap& mapV, dim3 grid,
                           cudaStream_t s) {
  switch (a.G) {
    case 1: return launch_split<D, 1>(a, mapK, mapV, grid, s);
    case 2: return launch_split<D, 2>(a, mapK, mapV, grid, s);
    case 3: return launch_split<D, 3>(a, mapK, mapV, grid, s);
    case 4: return launch_split<D, 4>(a, mapK, mapV, grid, s);
    case 5: return launch_split<D, 5>(a, mapK, mapV, grid, s);
    case 6: return launch_split<D, 6>(a, mapK, mapV, grid, s);
    case 7: return launch_split<D, 7>(a, mapK, mapV, grid, s);
    case 8: return launch_split<D, 8>(a, mapK, mapV, grid, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace
}  // namespace l2a

using namespace l2a;

extern "C" l2a_status l2a_decode_workspace_bytes(const l2a_params* p, size_t* ws_bytes) {
  size_t unused = 0;
  l2a_status st = l2a_workspace_bytes(p, &unused, nullptr, nullptr);
  if (st != L2A_OK) return st;
  if (!ws_bytes || p->Lq != 1) return L2A_ERR_INVALID_ARG;
  int nl, ng;
  plan_chunks(p, &nl, &ng);
  *ws_bytes = kWsHeaderBytes + align_up((size_t)p->B * p->Hq * (nl + ng) * (p->D + 2) * sizeof(float), 256);
  return L2A_OK;
}

extern "C" l2a_status l2a_decode(const l2a_params* p, const void* q, const void* K, const void* V, const uint8_t* d,
                                 void* O, void* ws, size_t ws_bytes, void* stream) {
  size_t need = 0;
  l2a_status st = l2a_decode_workspace_bytes(p, &need);
  if (st != L2A_OK) return st;
  if (!q || !K || !V || !O) return L2A_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V) |
       reinterpret_cast<uintptr_t>(O)) & 15)
    return L2A_ERR_INVALID_ARG;
  if (p->Hq / p->Hkv > kMaxGroup) return L2A_ERR_UNSUPPORTED;
  if (p->seq_bounds) return L2A_ERR_UNSUPPORTED;   // a decode step has one cache per batch entry
  if (p->q_pos_offset >= p->Lk) return L2A_ERR_INVALID_ARG;     // the new token's own key must be in the cache
  if (!ws || (reinterpret_cast<uintptr_t>(ws) % 256) != 0 || ws_bytes < need) return L2A_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(ws, 0, kWsHeaderBytes, s) != cudaSuccess) return L2A_ERR_CUDA;
  CUtensorMap mapK, mapV;
  if (!is_dense(p->q_stride, p->Lq, p->Hq * p->D) || !is_dense(p->o_stride, p->Lq, p->Hq * p->D)) return L2A_ERR_UNSUPPORTED;
  const RowStrides ks = resolve_strides(p->k_stride, p->Lk, p->Hkv * p->D);
  const RowStrides vs = resolve_strides(p->v_stride, p->Lk, p->Hkv * p->D);
  if (!encode_rows_map(&mapK, K, p->B, p->Lk, p->Hkv * p->D, kDecKeys, p->D, ks.b, ks.t) ||
      !encode_rows_map(&mapV, V, p->B, p->Lk, p->Hkv * p->D, kDecKeys, p->D, vs.b, vs.t))
    return L2A_ERR_CUDA;
  DecodeArgs a;
  a.B = p->B; a.Lk = p->Lk; a.Hq = p->Hq; a.Hkv = p->Hkv; a.G = p->Hq / p->Hkv;
  a.window = p->window;
  a.q_pos = p->q_pos_offset;
  a.scale_log2 = (p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->D)) * 1.4426950408889634f;
  plan_chunks(p, &a.n_loc, &a.n_glb);
  a.q = static_cast<const bf16*>(q);
  a.d = d;
  a.status = static_cast<int*>(ws);
  a.part = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + kWsHeaderBytes);
  a.O = static_cast<bf16*>(O);
  dim3 grid(a.n_loc + a.n_glb, p->Hkv, p->B);
  dim3 mgrid(p->Hq, p->B);
  cudaError_t e;
  if (p->D == 128) {
    e = launch_split_d<128>(a, mapK, mapV, grid, s);
    if (e == cudaSuccess) decode_merge_kernel<128><<<mgrid, 128, 0, s>>>(a);
  } else {
    e = launch_split_d<64>(a, mapK, mapV, grid, s);
    if (e == cudaSuccess) decode_merge_kernel<64><<<mgrid, 64, 0, s>>>(a);
  }
  if (e != cudaSuccess) return L2A_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? L2A_OK : L2A_ERR_CUDA;
}
