// Decode step of the layer (Section 3.4): one new query token per sequence attends to the last W+1 keys of the
// cache (Local Attention) and, only if its routing decision d = 1, to the whole cache (Global Attention);
// o = s + d * a.  The work is a pass over the K/V cache: HBM-bound.  The cache of every KV head is split into
// chunks processed by independent CTAs (flash-decoding style partial soft-max), merged by a second small kernel.
//
// Split kernel, one CTA = one chunk of keys of one (batch entry, KV head), for all G query heads of the group:
//   scores   : lane = key.  Each lane reads its key row (16-byte loads; neighbouring chunks of a row hit L1) and
//              accumulates the G dot products against q held in shared memory (broadcast reads).
//   soft-max : running maximum per head over the warp, exp2 domain.
//   P*V      : lane = 4 consecutive output columns.  One coalesced load per value row; each probability is
//              broadcast from its key's lane with a shuffle.
#include <math.h>

#include "l2a_common.cuh"

namespace l2a {

namespace {

constexpr int kDecThreads = 256;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kMaxGroup = 8;   // query heads per KV head supported by the decode kernels

struct DecodeArgs {
  int B, Lk, Hq, Hkv, G;
  int window, q_pos;       // the new token sits at position q_pos (normally Lk - 1)
  float scale_log2;
  int n_loc, n_glb;        // chunks of the local / global key range
  const bf16* q;           // [B, Hq, D]
  const bf16* K;           // [B, Lk, Hkv, D]
  const bf16* V;
  const uint8_t* d;        // [B] routing decision of the new token (NULL = never routed)
  float* part;             // [B, Hq, n_loc + n_glb, D + 2]  (acc[D], m, l)
  bf16* O;                 // [B, Hq, D]
};

__device__ __forceinline__ void chunk_range(int lo, int hi, int n, int i, int& c_lo, int& c_hi) {
  const int len = hi - lo + 1;
  int per = (len + n - 1) / n;
  per = (per + 31) / 32 * 32;
  c_lo = lo + i * per;
  c_hi = min(hi, c_lo + per - 1);
}

template <int D, int G>
__global__ void __launch_bounds__(kDecThreads, 2) decode_split_kernel(const DecodeArgs a) {
  constexpr int kPerLane = D / 32;                 // output columns per lane (4 or 2)
  const int item = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const bool glb = item >= a.n_loc;
  if (glb && (a.d == nullptr || a.d[b] == 0)) return;          // Global Attention is skipped when d = 0
  const int lo = glb ? 0 : max(0, a.q_pos - a.window);
  int c_lo, c_hi;
  chunk_range(lo, a.q_pos, glb ? a.n_glb : a.n_loc, glb ? item - a.n_loc : item, c_lo, c_hi);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  __shared__ __align__(16) float q_s[G * D];
  __shared__ float red_m[kDecWarps][G], red_l[kDecWarps][G];
  __shared__ __align__(16) float red_acc[kDecWarps][G][D];

  for (int i = tid; i < G * D; i += kDecThreads) {
    const int h = g * G + i / D;
    q_s[i] = __bfloat162float(a.q[((int64_t)b * a.Hq + h) * D + i % D]) * a.scale_log2;
  }
  __syncthreads();

  float m[G], l[G], acc[G][kPerLane];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    m[h] = -INFINITY;
    l[h] = 0.f;
#pragma unroll
    for (int e = 0; e < kPerLane; ++e) acc[h][e] = 0.f;
  }
  const int64_t row_stride = (int64_t)a.Hkv * D;
  const bf16* Kb = a.K + ((int64_t)b * a.Lk) * row_stride + (int64_t)g * D;
  const bf16* Vb = a.V + ((int64_t)b * a.Lk) * row_stride + (int64_t)g * D;

  for (int k0 = c_lo + warp * 32; k0 <= c_hi; k0 += kDecWarps * 32) {
    const int k = k0 + lane;
    const bool valid = k <= c_hi;
    // ---- scores of this lane's key against the G query heads
    float2 sc2[G];   // two partial sums per head (packed f32x2 FMAs)
#pragma unroll
    for (int h = 0; h < G; ++h) sc2[h] = make_float2(0.f, 0.f);
    {
      // every lane reads a row (lanes past the chunk re-read its last key; their scores are discarded), and all
      // 16-byte loads of the row are issued before the first one is used: 8 KB in flight per warp
      const uint4* krow = reinterpret_cast<const uint4*>(Kb + (int64_t)min(k, c_hi) * row_stride);
      uint4 kv[D / 8];
#pragma unroll
      for (int c = 0; c < D / 8; ++c) kv[c] = __ldg(&krow[c]);
#pragma unroll
      for (int c = 0; c < D / 8; ++c) {
        const uint32_t u[4] = {kv[c].x, kv[c].y, kv[c].z, kv[c].w};
        float kf[8];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          kf[2 * x] = __uint_as_float(u[x] << 16);
          kf[2 * x + 1] = __uint_as_float(u[x] & 0xffff0000u);
        }
#pragma unroll
        for (int h = 0; h < G; ++h) {
          const float4 qa = *reinterpret_cast<const float4*>(&q_s[h * D + c * 8]);
          const float4 qb = *reinterpret_cast<const float4*>(&q_s[h * D + c * 8 + 4]);
          sc2[h] = __ffma2_rn(make_float2(kf[0], kf[1]), make_float2(qa.x, qa.y), sc2[h]);
          sc2[h] = __ffma2_rn(make_float2(kf[2], kf[3]), make_float2(qa.z, qa.w), sc2[h]);
          sc2[h] = __ffma2_rn(make_float2(kf[4], kf[5]), make_float2(qb.x, qb.y), sc2[h]);
          sc2[h] = __ffma2_rn(make_float2(kf[6], kf[7]), make_float2(qb.z, qb.w), sc2[h]);
        }
      }
    }
    float sc[G];
#pragma unroll
    for (int h = 0; h < G; ++h) sc[h] = sc2[h].x + sc2[h].y;
    // ---- online soft-max over the 32 keys of this step
    float p[G];
#pragma unroll
    for (int h = 0; h < G; ++h) {
      {
        float mx = valid ? sc[h] : -INFINITY;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        const float m_new = fmaxf(m[h], mx);
        const float alpha = exp2f(m[h] - m_new);           // 0 on the first step (m = -inf)
        p[h] = valid ? exp2f(sc[h] - m_new) : 0.f;
        l[h] = l[h] * alpha + p[h];                        // per-lane partial sum, reduced at the end
#pragma unroll
        for (int e = 0; e < kPerLane; ++e) acc[h][e] *= alpha;
        m[h] = m_new;
      }
    }
    // ---- P * V: one coalesced value row per key, probabilities broadcast from the key's lane
    // (keys past the chunk have p = 0; their row index is clamped so that no branch is needed)
#pragma unroll 1
    for (int kk0 = 0; kk0 < 32; kk0 += 8) {
      if (k0 + kk0 > c_hi) break;
      uint32_t vraw[8][kPerLane / 2];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const bf16* vrow = Vb + (int64_t)min(k0 + kk0 + j, c_hi) * row_stride + lane * kPerLane;
        if constexpr (kPerLane == 4) {
          const uint2 vv = __ldg(reinterpret_cast<const uint2*>(vrow));
          vraw[j][0] = vv.x; vraw[j][1] = vv.y;
        } else {
          vraw[j][0] = __ldg(reinterpret_cast<const uint32_t*>(vrow));
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float vf[kPerLane];
#pragma unroll
        for (int x = 0; x < kPerLane / 2; ++x) {
          vf[2 * x] = __uint_as_float(vraw[j][x] << 16);
          vf[2 * x + 1] = __uint_as_float(vraw[j][x] & 0xffff0000u);
        }
#pragma unroll
        for (int h = 0; h < G; ++h) {
          const float ph = __shfl_sync(0xffffffffu, p[h], kk0 + j);
#pragma unroll
          for (int e = 0; e < kPerLane; e += 2) {
            const float2 r = __ffma2_rn(make_float2(ph, ph), make_float2(vf[e], vf[e + 1]), make_float2(acc[h][e], acc[h][e + 1]));
            acc[h][e] = r.x;
            acc[h][e + 1] = r.y;
          }
        }
      }
    }
  }

  // ---- merge the warps of this CTA, then write the chunk's partial result
#pragma unroll
  for (int h = 0; h < G; ++h) {
    {
      float ls = l[h];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, o);
      if (lane == 0) { red_m[warp][h] = m[h]; red_l[warp][h] = ls; }
#pragma unroll
      for (int e = 0; e < kPerLane; ++e) red_acc[warp][h][lane * kPerLane + e] = acc[h][e];
    }
  }
  __syncthreads();
  const int n_items = a.n_loc + a.n_glb;
  for (int i = tid; i < G * D; i += kDecThreads) {
    const int h = i / D, col = i % D;
    float M = -INFINITY;
    for (int w = 0; w < kDecWarps; ++w) M = fmaxf(M, red_m[w][h]);
    float L = 0.f, A = 0.f;
    for (int w = 0; w < kDecWarps; ++w) {
      const float f = (red_m[w][h] == -INFINITY) ? 0.f : exp2f(red_m[w][h] - M);
      L += red_l[w][h] * f;
      A += red_acc[w][h][col] * f;
    }
    float* dst = a.part + (((int64_t)b * a.Hq + g * G + h) * n_items + item) * (D + 2);
    dst[col] = A;
    if (col == 0) { dst[D] = M; dst[D + 1] = L; }
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
  // about 2048 keys per CTA over the cache and 1024 over the local window: thousands of CTAs at long context
  // (those of non-routed sequences exit at once), and the merge stays a few hundred partials per head
  const int pos = p->q_pos_offset;
  const int local_len = (pos < p->window ? pos : p->window) + 1;
  int ng = ceil_div(pos + 1, 2048);
  if (ng > 512) ng = 512;
  int nl = ceil_div(local_len, 1024);
  *n_loc = nl < 1 ? 1 : nl;
  *n_glb = ng < 1 ? 1 : ng;
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
  *ws_bytes = align_up((size_t)p->B * p->Hq * (nl + ng) * (p->D + 2) * sizeof(float), 256);
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
  if (!ws || (reinterpret_cast<uintptr_t>(ws) % 256) != 0 || ws_bytes < need) return L2A_ERR_WORKSPACE;
  DecodeArgs a;
  a.B = p->B; a.Lk = p->Lk; a.Hq = p->Hq; a.Hkv = p->Hkv; a.G = p->Hq / p->Hkv;
  a.window = p->window;
  a.q_pos = p->q_pos_offset;
  a.scale_log2 = (p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->D)) * 1.4426950408889634f;
  plan_chunks(p, &a.n_loc, &a.n_glb);
  a.q = static_cast<const bf16*>(q); a.K = static_cast<const bf16*>(K); a.V = static_cast<const bf16*>(V);
  a.d = d;
  a.part = static_cast<float*>(ws);
  a.O = static_cast<bf16*>(O);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  dim3 grid(a.n_loc + a.n_glb, p->Hkv, p->B);
  dim3 mgrid(p->Hq, p->B);
#define L2A_DECODE_CASE(DD, GG)                                                     \
  case GG: decode_split_kernel<DD, GG><<<grid, kDecThreads, 0, s>>>(a); break;
  if (p->D == 128) {
    switch (a.G) {
      L2A_DECODE_CASE(128, 1) L2A_DECODE_CASE(128, 2) L2A_DECODE_CASE(128, 3) L2A_DECODE_CASE(128, 4)
      L2A_DECODE_CASE(128, 5) L2A_DECODE_CASE(128, 6) L2A_DECODE_CASE(128, 7) L2A_DECODE_CASE(128, 8)
    }
    decode_merge_kernel<128><<<mgrid, 128, 0, s>>>(a);
  } else {
    switch (a.G) {
      L2A_DECODE_CASE(64, 1) L2A_DECODE_CASE(64, 2) L2A_DECODE_CASE(64, 3) L2A_DECODE_CASE(64, 4)
      L2A_DECODE_CASE(64, 5) L2A_DECODE_CASE(64, 6) L2A_DECODE_CASE(64, 7) L2A_DECODE_CASE(64, 8)
    }
    decode_merge_kernel<64><<<mgrid, 64, 0, s>>>(a);
  }
#undef L2A_DECODE_CASE
  return cudaGetLastError() == cudaSuccess ? L2A_OK : L2A_ERR_CUDA;
}
