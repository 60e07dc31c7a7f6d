// Router backward under the straight-through estimator (Section 3.3, Eq. 7): with d_hat_t = sigmoid(z_t),
//   dL/dd_hat_t = dgate_t + 2 c d_hat_t      (dgate_t = dL/do_t . a_t from the attention backward; c = lambda / (n L))
//   dz_t = dL/dd_hat_t * d_hat_t (1 - d_hat_t),   dW = sum_t dz_t s_t,   dbias = sum_t dz_t,
//   dL/ds_t = dL/do_t + dz_t W                    (o_t = s_t + d_t a_t, and z_t = W s_t + bias)
// One pass over S (and over dO when the combined gradient of s_t is wanted): HBM-bound.
// A CTA takes a contiguous range of tokens; a thread owns 8 columns of the Hq*D vector and keeps their dW partial
// sums in registers across the CTA's tokens, then adds them to dW with atomics.
#include "l2a_common.cuh"

namespace l2a {

namespace {

constexpr int kRbTokens = 64;        // tokens whose dz is staged in shared memory at a time
constexpr int kRbMaxThreads = 512;

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    f[2 * k] = __uint_as_float(u[k] << 16);
    f[2 * k + 1] = __uint_as_float(u[k] & 0xffff0000u);
  }
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// The grid is sized to the machine, not to the input: CTA i owns the contiguous token range
// [i * n / gridDim, (i + 1) * n / gridDim), so every CTA streams the same number of bytes (no partial last wave)
// and adds its dW partial sums once.
__global__ void __launch_bounds__(kRbMaxThreads)
router_backward_kernel(const bf16* __restrict__ S, const float* __restrict__ w, const float* __restrict__ logits,
                       const float* __restrict__ dgate, float coeff, const bf16* dO /* may alias dS */,
                       float* __restrict__ dz_out, float* __restrict__ dw, float* __restrict__ dbias,
                       bf16* dS, int64_t n_tokens, int row_elems) {
  __shared__ float dz_s[kRbTokens];
  const int tid = threadIdx.x;
  const int64_t t_begin = n_tokens * blockIdx.x / gridDim.x, t_end = n_tokens * (blockIdx.x + 1) / gridDim.x;
  const int n_chunks = row_elems / 8;
  bool first_pass = true;
  for (int chunk0 = 0; chunk0 < n_chunks; chunk0 += blockDim.x, first_pass = false) {
    const int chunk = chunk0 + tid;
    const bool active = chunk < n_chunks;
    float wv[8], acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) { wv[e] = 0.f; acc[e] = 0.f; }
    if (active) {
      const float4 wa = __ldg(reinterpret_cast<const float4*>(w) + 2 * chunk);
      const float4 wb = __ldg(reinterpret_cast<const float4*>(w) + 2 * chunk + 1);
      wv[0] = wa.x; wv[1] = wa.y; wv[2] = wa.z; wv[3] = wa.w; wv[4] = wb.x; wv[5] = wb.y; wv[6] = wb.z; wv[7] = wb.w;
    }
    for (int64_t token0 = t_begin; token0 < t_end; token0 += kRbTokens) {
      const int nt = (int)(t_end - token0 < kRbTokens ? t_end - token0 : kRbTokens);
      __syncthreads();                     // the previous block's dz values are no longer needed
      if (tid < kRbTokens) {               // whole warps
        float dz = 0.f;
        if (tid < nt) {
          const float z = logits[token0 + tid];
          const float d_hat = 1.0f / (1.0f + expf(-z));
          const float g = (dgate != nullptr ? dgate[token0 + tid] : 0.f) + 2.0f * coeff * d_hat;
          dz = g * d_hat * (1.0f - d_hat);
          if (dz_out != nullptr && first_pass) dz_out[token0 + tid] = dz;
        }
        dz_s[tid] = dz;
        if (dbias != nullptr && first_pass) {
          float sum = dz;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
          if ((tid & 31) == 0) atomicAdd(dbias, sum);
        }
      }
      __syncthreads();
      if (!active) continue;
      const uint4* S4 = reinterpret_cast<const uint4*>(S) + token0 * n_chunks + chunk;
      if (dS == nullptr) {
#pragma unroll 8
        for (int t = 0; t < nt; ++t) {
          float sv[8];
          unpack8(__ldg(&S4[(int64_t)t * n_chunks]), sv);
          const float dz = dz_s[t];
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[e] = fmaf(dz, sv[e], acc[e]);
        }
      } else {
        const uint4* dO4 = reinterpret_cast<const uint4*>(dO) + token0 * n_chunks + chunk;
        uint4* dS4 = reinterpret_cast<uint4*>(dS) + token0 * n_chunks + chunk;
#pragma unroll 8
        for (int t = 0; t < nt; ++t) {
          float sv[8], ov[8];
          unpack8(__ldg(&S4[(int64_t)t * n_chunks]), sv);
          unpack8(dO4[(int64_t)t * n_chunks], ov);   // plain load: dS may be written in place
          const float dz = dz_s[t];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            acc[e] = fmaf(dz, sv[e], acc[e]);
            ov[e] = fmaf(dz, wv[e], ov[e]);
          }
          dS4[(int64_t)t * n_chunks] =
              make_uint4(pack2(ov[0], ov[1]), pack2(ov[2], ov[3]), pack2(ov[4], ov[5]), pack2(ov[6], ov[7]));
        }
      }
    }
    if (dw != nullptr && active) {
#pragma unroll
      for (int e = 0; e < 8; ++e) atomicAdd(&dw[chunk * 8 + e], acc[e]);
    }
  }
}

}  // namespace

cudaError_t launch_router_backward(const bf16* S, const float* w, const float* logits, const float* dgate, float coeff,
                                   const bf16* dO, float* dz, float* dw, float* dbias, bf16* dS, int B, int L,
                                   int row_elems, cudaStream_t stream) {
  const int64_t n_tokens = (int64_t)B * L;
  const int n_chunks = row_elems / 8;
  int threads = (n_chunks + 31) / 32 * 32;                 // one 16-byte column chunk per thread where it fits
  if (threads > kRbMaxThreads) threads = kRbMaxThreads;
  if (threads < kRbTokens) threads = kRbTokens;
  int device = 0, sms = 148;
  if (cudaGetDevice(&device) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
  int per_sm = 0;   // one resident wave: every CTA of the grid runs at once and owns an equal share
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, router_backward_kernel, threads, 0) != cudaSuccess ||
      per_sm < 1)
    per_sm = 1;
  int64_t blocks = (int64_t)sms * per_sm;
  const int64_t max_blocks = (n_tokens + 15) / 16;         // at least 16 tokens per CTA
  if (blocks > max_blocks) blocks = max_blocks;
  if (blocks < 1) blocks = 1;
  router_backward_kernel<<<(unsigned)blocks, threads, 0, stream>>>(S, w, logits, dgate, coeff, dO, dz, dw, dbias, dS, n_tokens,
                                                            row_elems);
  return cudaGetLastError();
}

}  // namespace l2a
