// Backward of the layer for sm_100a.
//
// The paper states only that the backward computes gradients for active queries and reuses L_c and
// Q_idx (Section 3.2); the arithmetic is the vector-Jacobian product of the forward with the routing
// mask fixed.  For each attention X in {local, global}, with P = exp(scale*q.k - lse_X):
//     Delta_i = dO_i . out_X,i      dP_ij = dO_i . v_j      dS_ij = P_ij (dP_ij - Delta_i)
//     dV_j += P_ij dO_i             dK_j += scale dS_ij q_i  dQ_i += scale dS_ij k_j
// where "global" rows are the routed rows only.
//
// Kernels
//   bwd_delta_kernel : Delta_loc (all rows), Delta_glb (compact rows), optional dgate.  HBM bound.
//   bwd_dkv_kernel   : key/value-stationary.  One CTA owns a block of 128 keys of one KV head and
//                      walks every query tile that can see it -- local band tiles of the G query heads,
//                      then the compact routed tiles from the first one at or after the block -- and
//                      accumulates dK, dV in TMEM (no atomics, one bf16 store).  The scores are built
//                      transposed (keys on TMEM lanes) so P^T and dS^T feed the second pair of MMAs
//                      straight from TMEM.
//   bwd_dq_kernel    : query-stationary, the forward's iteration space; local mode writes dQ, global mode
//                      adds the routed rows' global term at their positions.
#include "l2a_common.cuh"
#include "sm100_prims.cuh"

namespace l2a {

namespace {

constexpr int kBoxBytes = 128 * 128;
constexpr float kLog2e = 1.4426950408889634f;

// ------------------------------------------------------------------------------------------------
// Delta / dgate preprocess: one warp per (b, t), looping over heads.
__global__ void __launch_bounds__(256) bwd_delta_kernel(const bf16* __restrict__ dO, const bf16* __restrict__ S,
                                                        const bf16* __restrict__ A_c,
                                                        const uint8_t* __restrict__ d_mask,
                                                        const int32_t* __restrict__ prefix, float* __restrict__ delta_loc,
                                                        float* __restrict__ delta_glb, float* __restrict__ dgate, int B,
                                                        int L, int Hq, int D) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= B * L) return;
  const int b = warp / L, t = warp % L;
  const bool routed = d_mask[(int64_t)b * L + t] != 0;
  const int c = routed ? prefix[(int64_t)b * (L + 1) + t] : 0;
  const int64_t row = ((int64_t)b * L + t) * Hq * D;
  const int64_t crow = ((int64_t)b * L + c) * Hq * D;
  const int per_lane = D / 32;  // 2 or 4 elements
  float gate = 0.f;
  for (int h = 0; h < Hq; ++h) {
    float dl = 0.f, dg = 0.f;
    const bf16* po = dO + row + (int64_t)h * D + lane * per_lane;
    const bf16* ps = S + row + (int64_t)h * D + lane * per_lane;
    const bf16* pa = A_c + crow + (int64_t)h * D + lane * per_lane;
    for (int e = 0; e < per_lane; e += 2) {
      const float2 o2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(po + e));
      const float2 s2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(ps + e));
      dl += o2.x * s2.x + o2.y * s2.y;
      if (routed) {
        const float2 a2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(pa + e));
        dg += o2.x * a2.x + o2.y * a2.y;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      dl += __shfl_xor_sync(0xffffffffu, dl, o);
      dg += __shfl_xor_sync(0xffffffffu, dg, o);
    }
    if (lane == 0) {
      delta_loc[((int64_t)b * Hq + h) * L + t] = dl;
      if (routed) delta_glb[((int64_t)b * Hq + h) * L + c] = dg;
    }
    gate += dg;
  }
  if (dgate != nullptr && lane == 0) dgate[(int64_t)b * L + t] = routed ? gate : 0.f;
}

// ------------------------------------------------------------------------------------------------
struct BwdArgs {
  int B, Lq, Lk, Hq, Hkv, D;
  int window, q_pos_offset;
  float scale, scale_log2;
  int global_mode;  // dq kernel only
  const int32_t* q_idx;
  const int32_t* n_routed;
  const int32_t* prefix;
  const float* lse_loc;    // [B,Hq,Lq] by row
  const float* lse_glb;    // [B,Hq,Lq] by compact row
  const float* delta_loc;  // same indexing
  const float* delta_glb;
  bf16* dQ;
  bf16* dK;
  bf16* dV;
  int* status;
};

// ================================================================================================
// dQ kernel: one 128-row query tile per CTA.
//   warps 0-3: P / dS computation and epilogue (thread = query row); warp 4: TMA; warp 5: MMA.
//   TMEM: S [0,128) | dP [128,256) | dQ [256,256+D).  dS (bf16) overwrites the first half of dP.
template <int D>
struct DqSmem {
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kQOff = 0;
  static constexpr int kDoOff = kTileBytes;
  static constexpr int kKOff = 2 * kTileBytes;
  static constexpr int kVOff = 4 * kTileBytes;
  static constexpr int kBarOff = 6 * kTileBytes;
  static constexpr int kTotal = kBarOff + 256 + 1024;
};
struct DqBarriers {
  uint64_t q_full;
  uint64_t k_full[2], k_empty[2], v_full[2], v_empty[2];
  uint64_t sdp_full, ds_full, final_bar;
  uint32_t tmem_base;
  int abort_flag;
};

template <int D>
__global__ void __launch_bounds__(192, 1)
bwd_dq_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapDO,
              const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV, const BwdArgs a) {
  using SM = DqSmem<D>;
  constexpr int kDBoxes = D / 64, kKSteps = D / 16;
  const int n_tiles = (a.Lq + kTileM - 1) / kTileM;
  const int h = blockIdx.x % a.Hq;
  const int rest = blockIdx.x / a.Hq;
  const int b = rest % a.B;
  const int ti = n_tiles - 1 - rest / a.B;
  const int g = h / (a.Hq / a.Hkv);
  const int n_rows = a.global_mode ? a.n_routed[b] : a.Lq;
  const int row0 = ti * kTileM;
  if (row0 >= n_rows) return;
  const int32_t* q_idx_b = a.q_idx + (int64_t)b * a.Lq;
  const int w_eff = a.global_mode ? 0x3fffffff : a.window;
  const int last = min(row0 + kTileM - 1, n_rows - 1);
  const int min_pos = (a.global_mode ? q_idx_b[row0] : row0) + a.q_pos_offset;
  const int max_pos = (a.global_mode ? q_idx_b[last] : last) + a.q_pos_offset;
  const int jlo = (min_pos - w_eff > 0) ? (min_pos - w_eff) / kTileN : 0;
  const int jhi = max_pos / kTileN;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem + SM::kQOff;
  uint8_t* sDO = smem + SM::kDoOff;
  uint8_t* sK = smem + SM::kKOff;
  uint8_t* sV = smem + SM::kVOff;
  DqBarriers* bar = reinterpret_cast<DqBarriers*>(smem + SM::kBarOff);
  volatile int* abort_flag = &bar->abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    mbar_init(&bar->q_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bar->k_full[s], 1); mbar_init(&bar->k_empty[s], 1);
      mbar_init(&bar->v_full[s], 1); mbar_init(&bar->v_empty[s], 1);
    }
    mbar_init(&bar->sdp_full, 1);
    mbar_init(&bar->ds_full, 128);
    mbar_init(&bar->final_bar, 1);
    bar->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 5) { tmem_alloc(&bar->tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bar->tmem_base;

  if (warp == 4) {
    if (lane == 0) {
      tma_prefetch_desc(&mapQ); tma_prefetch_desc(&mapDO); tma_prefetch_desc(&mapK); tma_prefetch_desc(&mapV);
      mbar_expect_tx(&bar->q_full, 2 * SM::kTileBytes);
      for (int x = 0; x < kDBoxes; ++x) {
        tma_load_3d(sQ + x * kBoxBytes, &mapQ, &bar->q_full, h * D + x * 64, row0, b);
        tma_load_3d(sDO + x * kBoxBytes, &mapDO, &bar->q_full, h * D + x * 64, row0, b);
      }
      for (int j = jlo; j <= jhi; ++j) {
        const int it = j - jlo, s = it & 1;
        const uint32_t ph = (it >> 1) & 1;
        if (!mbar_wait(&bar->k_empty[s], ph ^ 1, abort_flag)) break;
        mbar_expect_tx(&bar->k_full[s], SM::kTileBytes);
        for (int x = 0; x < kDBoxes; ++x)
          tma_load_3d(sK + s * SM::kTileBytes + x * kBoxBytes, &mapK, &bar->k_full[s], g * D + x * 64, j * kTileN, b);
        if (!mbar_wait(&bar->v_empty[s], ph ^ 1, abort_flag)) break;
        mbar_expect_tx(&bar->v_full[s], SM::kTileBytes);
        for (int x = 0; x < kDBoxes; ++x)
          tma_load_3d(sV + s * SM::kTileBytes + x * kBoxBytes, &mapV, &bar->v_full[s], g * D + x * 64, j * kTileN, b);
      }
    }
    __syncwarp();
  } else if (warp == 5) {
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0);
      constexpr uint32_t idesc_dq = idesc_bf16_f32(128, D, 0, 1);
      bool ok = mbar_wait(&bar->q_full, 0, abort_flag);
      const uint32_t qa = smem_u32(sQ), doa = smem_u32(sDO);
      for (int j = jlo; ok && j <= jhi; ++j) {
        const int it = j - jlo, s = it & 1;
        const uint32_t ph = (it >> 1) & 1;
        if (!mbar_wait(&bar->k_full[s], ph, abort_flag) || !mbar_wait(&bar->v_full[s], ph, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t ka = smem_u32(sK + s * SM::kTileBytes), va = smem_u32(sV + s * SM::kTileBytes);
#pragma unroll
        for (int kk = 0; kk < kKSteps; ++kk) {
          const uint32_t off = (kk >> 2) * kBoxBytes + (kk & 3) * 32;
          mma_ss(tmem, smem_desc_sw128(qa + off, 16, 1024), smem_desc_sw128(ka + off, 16, 1024), idesc_s, kk > 0);
        }
#pragma unroll
        for (int kk = 0; kk < kKSteps; ++kk) {
          const uint32_t off = (kk >> 2) * kBoxBytes + (kk & 3) * 32;
          mma_ss(tmem + 128, smem_desc_sw128(doa + off, 16, 1024), smem_desc_sw128(va + off, 16, 1024), idesc_s, kk > 0);
        }
        tc_commit(&bar->sdp_full);
        tc_commit(&bar->v_empty[s]);
        if (!mbar_wait(&bar->ds_full, it & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < kTileN / 16; ++kk)
          mma_ts(tmem + 256, tmem + 128 + kk * 8, smem_desc_sw128(ka + kk * 2048, kBoxBytes, 1024), idesc_dq,
                 (j > jlo) || (kk > 0));
        tc_commit(&bar->k_empty[s]);
      }
      if (ok) tc_commit(&bar->final_bar);
    }
    __syncwarp();
  } else {
    const int r = warp * 32 + lane;
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    const int row = row0 + r;
    const bool valid = row < n_rows;
    const int seq_row = valid ? (a.global_mode ? q_idx_b[row] : row) : -1;
    const int pos = valid ? seq_row + a.q_pos_offset : -1;
    const int pos_lo = valid ? pos - w_eff : 0x7fffffff;
    const int64_t stat_idx = ((int64_t)b * a.Hq + h) * a.Lq + (valid ? row : 0);
    const float lse2 = valid ? (a.global_mode ? a.lse_glb : a.lse_loc)[stat_idx] * kLog2e : 0.f;
    const float delta = valid ? (a.global_mode ? a.delta_glb : a.delta_loc)[stat_idx] : 0.f;
    bool ok = true;
    for (int j = jlo; j <= jhi; ++j) {
      const int it = j - jlo;
      if (!__all_sync(0xffffffffu, mbar_wait(&bar->sdp_full, it & 1, abort_flag))) { ok = false; break; }
      tc_fence_after();
      const int k0 = j * kTileN;
      const bool partial = (k0 + kTileN - 1 > min_pos) || (k0 < max_pos - w_eff) || (last - row0 + 1 < kTileM);
#pragma unroll
      for (int c = 0; c < 2; ++c) {       // 64 keys at a time
        uint32_t sv[2][32], dv[2][32];
        tmem_ld32(tmem + lane_base + c * 64, sv[0]);
        tmem_ld32(tmem + lane_base + c * 64 + 32, sv[1]);
        tmem_ld32(tmem + lane_base + 128 + c * 64, dv[0]);
        tmem_ld32(tmem + lane_base + 128 + c * 64 + 32, dv[1]);
        tmem_ld_wait();
        if (c == 1) {
          // all of dP has been read: from here on the dS stores may overwrite its first half
        }
        uint32_t pk[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          float ds2[2];
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int idx = 2 * e + u;          // key within this 64-wide chunk
            const float sc = __uint_as_float(sv[idx >> 5][idx & 31]);
            const float dp = __uint_as_float(dv[idx >> 5][idx & 31]);
            float p = fast_exp2(fmaf(sc, a.scale_log2, -lse2));
            float ds = p * (dp - delta);
            if (partial) {
              const int kp = k0 + c * 64 + idx;
              if (!(kp <= pos && kp >= pos_lo)) ds = 0.f;
            }
            ds2[u] = ds;
          }
          pk[e] = pack_bf16(ds2[0], ds2[1]);
        }
        // dS chunk c -> packed columns [128 + 32c, 128 + 32c + 32).  Chunk 0 overwrites dP columns 0..31,
        // which were read above; chunk 1 overwrites dP columns 32..63, read in chunk 0's loads as well.
        if (c == 0) {
          // keep chunk 0's packed values until chunk 1's dP loads (columns 64..127) are done: the stores
          // only touch columns < 64 of dP, already consumed by this thread.
        }
        tmem_st32(tmem + lane_base + 128 + c * 32, pk);
      }
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(&bar->ds_full);
    }
    if (ok && __all_sync(0xffffffffu, mbar_wait(&bar->final_bar, 0, abort_flag))) {
      tc_fence_after();
      bf16* dst = valid ? a.dQ + (((int64_t)b * a.Lq + seq_row) * a.Hq + h) * D : nullptr;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t v[32];
        tmem_ld32(tmem + lane_base + 256 + c * 32, v);
        tmem_ld_wait();
        if (dst) {
          float f[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) f[e] = __uint_as_float(v[e]) * a.scale;
          uint4* d4 = reinterpret_cast<uint4*>(dst + c * 32);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            if (a.global_mode) {
              const uint4 old = d4[q];
              const uint32_t ow[4] = {old.x, old.y, old.z, old.w};
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                f[8 * q + 2 * k] += __uint_as_float(ow[k] << 16);
                f[8 * q + 2 * k + 1] += __uint_as_float(ow[k] & 0xffff0000u);
              }
            }
            d4[q] = make_uint4(pack_bf16(f[8 * q], f[8 * q + 1]), pack_bf16(f[8 * q + 2], f[8 * q + 3]),
                               pack_bf16(f[8 * q + 4], f[8 * q + 5]), pack_bf16(f[8 * q + 6], f[8 * q + 7]));
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (bar->abort_flag) {
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    if (tid == 0) atomicExch(a.status, 1);
    __syncthreads();
  }
  if (warp == 5) tmem_dealloc(tmem, 512);
}

// ================================================================================================
// dK/dV kernel: one block of 128 keys of one KV head per CTA.
//   warps 0-3: P^T / dS^T computation and epilogue (thread = key); warp 4: TMA + per-item row
//   statistics staging; warp 5: MMA.
//   TMEM: S^T [0,128) | dP^T [128,256) | dV [256,256+D) | dK [256+D, 256+2D).
template <int D>
struct DkvSmem {
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kKOff = 0;
  static constexpr int kVOff = kTileBytes;
  static constexpr int kQOff = 2 * kTileBytes;       // 2 stages
  static constexpr int kDoOff = 4 * kTileBytes;      // 2 stages
  static constexpr int kStatOff = 6 * kTileBytes;    // 2 stages x {lse2[128], delta[128], pos[128], flags[4]}
  static constexpr int kStatStage = (3 * 128 + 4) * 4;
  static constexpr int kBarOff = kStatOff + 2 * kStatStage + 16;
  static constexpr int kTotal = kBarOff + 256 + 1024;
};
struct DkvBarriers {
  uint64_t kv_full;
  uint64_t qdo_full[2], qdo_empty[2];
  uint64_t sdp_full, pds_full, final_bar;
  uint32_t tmem_base;
  int abort_flag;
};

struct ItemPlan {
  int loc_t0, loc_nt;   // first local query tile, number of local tiles
  int glb_t0, glb_nt;   // first compact tile, number of compact tiles
  int per_head;         // loc_nt + glb_nt
  int total;            // per_head * G
};

__device__ __forceinline__ ItemPlan make_plan(const BwdArgs& a, int b, int k0) {
  ItemPlan p;
  // local: rows t with position in [k0, k0 + 127 + W]
  int tmin = k0 - a.q_pos_offset;
  const long long tmax_ll = (long long)k0 + kTileN - 1 + a.window - a.q_pos_offset;
  int tmax = tmax_ll > a.Lq - 1 ? a.Lq - 1 : (int)tmax_ll;
  if (tmin < 0) tmin = 0;
  if (tmax < tmin) { p.loc_t0 = 0; p.loc_nt = 0; }
  else { p.loc_t0 = tmin / kTileM; p.loc_nt = tmax / kTileM - p.loc_t0 + 1; }
  // global: compact rows whose position is >= k0
  const int n_c = a.n_routed[b];
  if (tmin > a.Lq - 1 || n_c == 0) { p.glb_t0 = 0; p.glb_nt = 0; }
  else {
    const int c_min = a.prefix[(int64_t)b * (a.Lq + 1) + tmin];
    if (c_min >= n_c) { p.glb_t0 = 0; p.glb_nt = 0; }
    else { p.glb_t0 = c_min / kTileM; p.glb_nt = (n_c - 1) / kTileM - p.glb_t0 + 1; }
  }
  p.per_head = p.loc_nt + p.glb_nt;
  p.total = p.per_head * (a.Hq / a.Hkv);
  return p;
}

template <int D>
__global__ void __launch_bounds__(192, 1)
bwd_dkv_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapDO,
               const __grid_constant__ CUtensorMap mapQc, const __grid_constant__ CUtensorMap mapDOc,
               const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV, const BwdArgs a) {
  using SM = DkvSmem<D>;
  constexpr int kDBoxes = D / 64, kKSteps = D / 16;
  const int n_kblocks = (a.Lk + kTileN - 1) / kTileN;
  // key blocks ascending (most work first) inside one KV head; KV heads outermost so that the CTAs
  // running together share the same query tiles in L2
  const int j = blockIdx.x % n_kblocks;
  const int rest = blockIdx.x / n_kblocks;
  const int b = rest % a.B;
  const int g = rest / a.B;
  const int G = a.Hq / a.Hkv;
  const int k0 = j * kTileN;
  const ItemPlan plan = make_plan(a, b, k0);
  const int n_c = a.n_routed[b];

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sK = smem + SM::kKOff;
  uint8_t* sV = smem + SM::kVOff;
  uint8_t* sQ = smem + SM::kQOff;
  uint8_t* sDO = smem + SM::kDoOff;
  DkvBarriers* bar = reinterpret_cast<DkvBarriers*>(smem + SM::kBarOff);
  volatile int* abort_flag = &bar->abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (plan.total == 0) {
    // no query can see these keys: their gradients are zero
    for (int i = tid; i < kTileN * (D / 8); i += blockDim.x) {
      const int kr = i / (D / 8), c8 = i % (D / 8);
      if (k0 + kr < a.Lk) {
        const int64_t o = (((int64_t)b * a.Lk + k0 + kr) * a.Hkv + g) * D + c8 * 8;
        *reinterpret_cast<uint4*>(a.dK + o) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(a.dV + o) = make_uint4(0, 0, 0, 0);
      }
    }
    return;
  }

  if (tid == 0) {
    mbar_init(&bar->kv_full, 1);
    for (int s = 0; s < 2; ++s) { mbar_init(&bar->qdo_full[s], 33); mbar_init(&bar->qdo_empty[s], 1); }
    mbar_init(&bar->sdp_full, 1);
    mbar_init(&bar->pds_full, 128);
    mbar_init(&bar->final_bar, 1);
    bar->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 5) { tmem_alloc(&bar->tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bar->tmem_base;

  // item i -> (head, mode, tile)
  auto decode = [&](int i, int& h, int& glb, int& tile) {
    const int hh = i / plan.per_head, r = i % plan.per_head;
    h = g * G + hh;
    if (r < plan.loc_nt) { glb = 0; tile = plan.loc_t0 + r; }
    else { glb = 1; tile = plan.glb_t0 + (r - plan.loc_nt); }
  };

  if (warp == 4) {
    // ------------------------------------------------------------------ producer: TMA + statistics
    if (lane == 0) {
      tma_prefetch_desc(&mapQ); tma_prefetch_desc(&mapDO); tma_prefetch_desc(&mapQc); tma_prefetch_desc(&mapDOc);
      mbar_expect_tx(&bar->kv_full, 2 * SM::kTileBytes);
      for (int x = 0; x < kDBoxes; ++x) {
        tma_load_3d(sK + x * kBoxBytes, &mapK, &bar->kv_full, g * D + x * 64, k0, b);
        tma_load_3d(sV + x * kBoxBytes, &mapV, &bar->kv_full, g * D + x * 64, k0, b);
      }
    }
    bool ok = true;
    for (int i = 0; i < plan.total; ++i) {
      const int s = i & 1;
      const uint32_t ph = (i >> 1) & 1;
      int h, glb, tile;
      decode(i, h, glb, tile);
      const int row0 = tile * kTileM;
      if (!__all_sync(0xffffffffu, mbar_wait(&bar->qdo_empty[s], ph ^ 1, abort_flag))) { ok = false; break; }
      if (lane == 0) {
        mbar_expect_tx(&bar->qdo_full[s], 2 * SM::kTileBytes);
        for (int x = 0; x < kDBoxes; ++x) {
          tma_load_3d(sQ + s * SM::kTileBytes + x * kBoxBytes, glb ? &mapQc : &mapQ, &bar->qdo_full[s],
                      h * D + x * 64, row0, b);
          tma_load_3d(sDO + s * SM::kTileBytes + x * kBoxBytes, glb ? &mapDOc : &mapDO, &bar->qdo_full[s],
                      h * D + x * 64, row0, b);
        }
      }
      float* st_lse = reinterpret_cast<float*>(smem + SM::kStatOff + s * SM::kStatStage);
      float* st_delta = st_lse + 128;
      int* st_pos = reinterpret_cast<int*>(st_delta + 128);
      int* st_flags = st_pos + 128;
      const int n_rows = glb ? n_c : a.Lq;
      const float* lse = glb ? a.lse_glb : a.lse_loc;
      const float* dl = glb ? a.delta_glb : a.delta_loc;
      int pmin = 0x7fffffff, pmax = -1, all_valid = 1;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int col = q * 32 + lane, row = row0 + col;
        const bool valid = row < n_rows;
        const int64_t si = ((int64_t)b * a.Hq + h) * a.Lq + (valid ? row : 0);
        st_lse[col] = valid ? lse[si] * kLog2e : 0.f;
        st_delta[col] = valid ? dl[si] : 0.f;
        const int pos = valid ? (glb ? a.q_idx[(int64_t)b * a.Lq + row] : row) + a.q_pos_offset : -1;
        st_pos[col] = pos;
        if (valid) { pmin = min(pmin, pos); pmax = max(pmax, pos); } else all_valid = 0;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        pmin = min(pmin, __shfl_xor_sync(0xffffffffu, pmin, o));
        pmax = max(pmax, __shfl_xor_sync(0xffffffffu, pmax, o));
        all_valid &= __shfl_xor_sync(0xffffffffu, all_valid, o);
      }
      if (lane == 0) {
        const int w_eff = glb ? 0x3fffffff : a.window;
        const int interior = all_valid && (k0 + kTileN - 1 <= pmin) && (k0 >= pmax - w_eff);
        st_flags[0] = interior ? 0 : 1;     // 1 = apply the element mask
        st_flags[1] = glb;
      }
      __syncwarp();
      mbar_arrive(&bar->qdo_full[s]);
    }
    (void)ok;
  } else if (warp == 5) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0);
      constexpr uint32_t idesc_acc = idesc_bf16_f32(128, D, 0, 1);
      bool ok = mbar_wait(&bar->kv_full, 0, abort_flag);
      const uint32_t ka = smem_u32(sK), va = smem_u32(sV);
      for (int i = 0; ok && i < plan.total; ++i) {
        const int s = i & 1;
        const uint32_t ph = (i >> 1) & 1;
        if (!mbar_wait(&bar->qdo_full[s], ph, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t qa = smem_u32(sQ + s * SM::kTileBytes), doa = smem_u32(sDO + s * SM::kTileBytes);
#pragma unroll
        for (int kk = 0; kk < kKSteps; ++kk) {   // S^T = K Q^T
          const uint32_t off = (kk >> 2) * kBoxBytes + (kk & 3) * 32;
          mma_ss(tmem, smem_desc_sw128(ka + off, 16, 1024), smem_desc_sw128(qa + off, 16, 1024), idesc_s, kk > 0);
        }
#pragma unroll
        for (int kk = 0; kk < kKSteps; ++kk) {   // dP^T = V dO^T
          const uint32_t off = (kk >> 2) * kBoxBytes + (kk & 3) * 32;
          mma_ss(tmem + 128, smem_desc_sw128(va + off, 16, 1024), smem_desc_sw128(doa + off, 16, 1024), idesc_s, kk > 0);
        }
        tc_commit(&bar->sdp_full);
        if (!mbar_wait(&bar->pds_full, i & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < kTileM / 16; ++kk)   // dV += P^T dO
          mma_ts(tmem + 256, tmem + kk * 8, smem_desc_sw128(doa + kk * 2048, kBoxBytes, 1024), idesc_acc,
                 (i > 0) || (kk > 0));
#pragma unroll
        for (int kk = 0; kk < kTileM / 16; ++kk)   // dK += dS^T Q
          mma_ts(tmem + 256 + D, tmem + 128 + kk * 8, smem_desc_sw128(qa + kk * 2048, kBoxBytes, 1024), idesc_acc,
                 (i > 0) || (kk > 0));
        tc_commit(&bar->qdo_empty[s]);
      }
      if (ok) tc_commit(&bar->final_bar);
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ P^T / dS^T and epilogue
    const int kr = warp * 32 + lane;           // key inside the block == TMEM lane
    const int kp = k0 + kr;
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    bool ok = true;
    for (int i = 0; i < plan.total; ++i) {
      const int s = i & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(&bar->sdp_full, i & 1, abort_flag))) { ok = false; break; }
      tc_fence_after();
      const float* st_lse = reinterpret_cast<const float*>(smem + SM::kStatOff + s * SM::kStatStage);
      const float* st_delta = st_lse + 128;
      const int* st_pos = reinterpret_cast<const int*>(st_delta + 128);
      const int* st_flags = st_pos + 128;
      const bool masked = st_flags[0] != 0;
      const int w_eff = st_flags[1] ? 0x3fffffff : a.window;
#pragma unroll
      for (int c = 0; c < 2; ++c) {   // 64 query columns at a time
        uint32_t sv[2][32], dv[2][32];
        tmem_ld32(tmem + lane_base + c * 64, sv[0]);
        tmem_ld32(tmem + lane_base + c * 64 + 32, sv[1]);
        tmem_ld32(tmem + lane_base + 128 + c * 64, dv[0]);
        tmem_ld32(tmem + lane_base + 128 + c * 64 + 32, dv[1]);
        tmem_ld_wait();
        uint32_t pp[32], pd[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          float p2[2], ds2[2];
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int idx = 2 * e + u, col = c * 64 + idx;
            const float sc = __uint_as_float(sv[idx >> 5][idx & 31]);
            const float dp = __uint_as_float(dv[idx >> 5][idx & 31]);
            float p = fast_exp2(fmaf(sc, a.scale_log2, -st_lse[col]));
            float ds = p * (dp - st_delta[col]);
            if (masked) {
              const int pos = st_pos[col];
              if (!(kp <= pos && kp >= pos - w_eff)) { p = 0.f; ds = 0.f; }
            }
            p2[u] = p; ds2[u] = ds;
          }
          pp[e] = pack_bf16(p2[0], p2[1]);
          pd[e] = pack_bf16(ds2[0], ds2[1]);
        }
        // P^T chunk c -> S^T columns [32c, 32c+32); dS^T chunk c -> dP^T columns [32c, 32c+32): both ranges
        // lie inside the columns this thread has already loaded (chunk 0 reads 0..63, chunk 1 reads 64..127)
        tmem_st32(tmem + lane_base + c * 32, pp);
        tmem_st32(tmem + lane_base + 128 + c * 32, pd);
      }
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(&bar->pds_full);
    }
    if (ok && __all_sync(0xffffffffu, mbar_wait(&bar->final_bar, 0, abort_flag))) {
      tc_fence_after();
      const bool valid = kp < a.Lk;
      const int64_t o = (((int64_t)b * a.Lk + (valid ? kp : 0)) * a.Hkv + g) * D;
#pragma unroll
      for (int which = 0; which < 2; ++which) {
        bf16* dst = (which == 0 ? a.dV : a.dK) + o;
        const float mul = which == 0 ? 1.0f : a.scale;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t v[32];
          tmem_ld32(tmem + lane_base + 256 + which * D + c * 32, v);
          tmem_ld_wait();
          if (valid) {
            uint4* d4 = reinterpret_cast<uint4*>(dst + c * 32);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              float f[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[8 * q + e]) * mul;
              d4[q] = make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]),
                                 pack_bf16(f[6], f[7]));
            }
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (bar->abort_flag) {
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    if (tid == 0) atomicExch(a.status, 1);
    __syncthreads();
  }
  if (warp == 5) tmem_dealloc(tmem, 512);
}

size_t rows_bytes(const l2a_params* p) { return align_up((size_t)p->B * p->Lq * p->Hq * p->D * sizeof(bf16), 256); }
size_t stat_bytes(const l2a_params* p) { return align_up((size_t)p->B * p->Hq * p->Lq * sizeof(float), 256); }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

template <int D>
cudaError_t launch_bwd_kernels(const BwdArgs& base, const CUtensorMap& mapQ, const CUtensorMap& mapDO,
                               const CUtensorMap& mapQc, const CUtensorMap& mapDOc, const CUtensorMap& mapK,
                               const CUtensorMap& mapV, cudaStream_t s) {
  cudaError_t e;
  e = cudaFuncSetAttribute(bwd_dkv_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, DkvSmem<D>::kTotal);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(bwd_dq_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, DqSmem<D>::kTotal);
  if (e != cudaSuccess) return e;
  const unsigned n_kblocks = (base.Lk + kTileN - 1) / kTileN;
  bwd_dkv_kernel<D><<<n_kblocks * base.B * base.Hkv, 192, DkvSmem<D>::kTotal, s>>>(mapQ, mapDO, mapQc, mapDOc, mapK,
                                                                                  mapV, base);
  phase_events().mark(s);
  const unsigned n_tiles = (base.Lq + kTileM - 1) / kTileM;
  BwdArgs a = base;
  a.global_mode = 0;
  bwd_dq_kernel<D><<<n_tiles * base.B * base.Hq, 192, DqSmem<D>::kTotal, s>>>(mapQ, mapDO, mapK, mapV, a);
  phase_events().mark(s);
  a.global_mode = 1;
  bwd_dq_kernel<D><<<n_tiles * base.B * base.Hq, 192, DqSmem<D>::kTotal, s>>>(mapQc, mapDOc, mapK, mapV, a);
  phase_events().mark(s);
  return cudaGetLastError();
}

}  // namespace

size_t bwd_ws_size(const l2a_params* p) { return kWsHeaderBytes + 2 * rows_bytes(p) + 2 * stat_bytes(p); }

}  // namespace l2a

using namespace l2a;

extern "C" l2a_status l2a_backward(const l2a_params* p, const void* Q, const void* K, const void* V,
                                   const uint8_t* d_mask, const int32_t* q_idx, const int32_t* n_routed,
                                   const int32_t* prefix, const void* dO, const void* S_save, const void* A_c,
                                   const float* lse_loc, const float* lse_glb, void* dQ, void* dK, void* dV,
                                   float* dgate, void* bwd_ws, size_t bwd_ws_bytes, void* stream) {
  if (!p) return L2A_ERR_INVALID_ARG;
  size_t need = 0;
  l2a_status st = l2a_workspace_bytes(p, nullptr, nullptr, &need);
  if (st != L2A_OK) return st;
  if (p->flags & (L2A_FLAG_SKIP_LOCAL | L2A_FLAG_SKIP_GLOBAL)) return L2A_ERR_UNSUPPORTED;
  if (!Q || !K || !V || !d_mask || !q_idx || !n_routed || !prefix || !dO || !S_save || !A_c || !lse_loc || !lse_glb ||
      !dQ || !dK || !dV)
    return L2A_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(dO) || !aligned16(S_save) || !aligned16(A_c) ||
      !aligned16(dQ) || !aligned16(dK) || !aligned16(dV))
    return L2A_ERR_INVALID_ARG;
  if (!bwd_ws || (reinterpret_cast<uintptr_t>(bwd_ws) % 256) != 0 || bwd_ws_bytes < need) return L2A_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(bwd_ws);
  if (cudaMemsetAsync(ws, 0, kWsHeaderBytes, s) != cudaSuccess) return L2A_ERR_CUDA;
  bf16* Qc = reinterpret_cast<bf16*>(ws + kWsHeaderBytes);
  bf16* dOc = reinterpret_cast<bf16*>(ws + kWsHeaderBytes + rows_bytes(p));
  float* delta_loc = reinterpret_cast<float*>(ws + kWsHeaderBytes + 2 * rows_bytes(p));
  float* delta_glb = reinterpret_cast<float*>(ws + kWsHeaderBytes + 2 * rows_bytes(p) + stat_bytes(p));

  CUtensorMap mapQ, mapDO, mapQc, mapDOc, mapK, mapV;
  if (!encode_rows_map(&mapQ, Q, p->B, p->Lq, p->Hq * p->D, kTileM) ||
      !encode_rows_map(&mapDO, dO, p->B, p->Lq, p->Hq * p->D, kTileM) ||
      !encode_rows_map(&mapQc, Qc, p->B, p->Lq, p->Hq * p->D, kTileM) ||
      !encode_rows_map(&mapDOc, dOc, p->B, p->Lq, p->Hq * p->D, kTileM) ||
      !encode_rows_map(&mapK, K, p->B, p->Lk, p->Hkv * p->D, kTileN) ||
      !encode_rows_map(&mapV, V, p->B, p->Lk, p->Hkv * p->D, kTileN))
    return L2A_ERR_CUDA;

  PhaseEvents& pe = phase_events();
  struct ClearOnExit { PhaseEvents& p; ~ClearOnExit() { p.clear(); } } clear_on_exit{pe};
  pe.mark(s);
  if (launch_gather_rows(static_cast<const bf16*>(Q), Qc, q_idx, n_routed, p->B, p->Lq, p->Hq * p->D, s) != cudaSuccess)
    return L2A_ERR_CUDA;
  if (launch_gather_rows(static_cast<const bf16*>(dO), dOc, q_idx, n_routed, p->B, p->Lq, p->Hq * p->D, s) !=
      cudaSuccess)
    return L2A_ERR_CUDA;
  pe.mark(s);
  {
    const int64_t warps = (int64_t)p->B * p->Lq;
    const unsigned blocks = (unsigned)((warps * 32 + 255) / 256);
    bwd_delta_kernel<<<blocks, 256, 0, s>>>(static_cast<const bf16*>(dO), static_cast<const bf16*>(S_save),
                                            static_cast<const bf16*>(A_c), d_mask, prefix, delta_loc, delta_glb, dgate,
                                            p->B, p->Lq, p->Hq, p->D);
    if (cudaGetLastError() != cudaSuccess) return L2A_ERR_CUDA;
  }
  pe.mark(s);
  BwdArgs a;
  a.B = p->B; a.Lq = p->Lq; a.Lk = p->Lk; a.Hq = p->Hq; a.Hkv = p->Hkv; a.D = p->D;
  a.window = p->window;
  a.q_pos_offset = p->q_pos_offset;
  a.scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->D);
  a.scale_log2 = a.scale * kLog2e;
  a.global_mode = 0;
  a.q_idx = q_idx; a.n_routed = n_routed; a.prefix = prefix;
  a.lse_loc = lse_loc; a.lse_glb = lse_glb; a.delta_loc = delta_loc; a.delta_glb = delta_glb;
  a.dQ = static_cast<bf16*>(dQ); a.dK = static_cast<bf16*>(dK); a.dV = static_cast<bf16*>(dV);
  a.status = reinterpret_cast<int*>(ws);
  cudaError_t e = p->D == 128 ? launch_bwd_kernels<128>(a, mapQ, mapDO, mapQc, mapDOc, mapK, mapV, s)
                              : launch_bwd_kernels<64>(a, mapQ, mapDO, mapQc, mapDOc, mapK, mapV, s);
  return e == cudaSuccess ? L2A_OK : L2A_ERR_CUDA;
}
