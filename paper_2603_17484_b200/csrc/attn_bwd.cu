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
//   dq_zero_kernel   : clears the fp32 dQ accumulators.
//   bwd_kernel       : key/value-stationary, five GEMMs per (query tile, key block) pair.  One CTA owns a block of
//                      128 keys of one KV head and walks every query tile that can see it -- local band tiles of
//                      the G query heads, then the compact routed tiles from the first one at or after the block.
//                      dK, dV accumulate in TMEM (no atomics, one bf16 store); the scores are built transposed (keys
//                      on TMEM lanes) so that P^T feeds dV straight from TMEM; dQ(i) = dS(i) K is a fresh tile per
//                      item that dedicated read-out warps add into fp32 accumulators in global memory.
//   dq_merge_kernel  : dQ = scale * (local accumulator + routed rows' global accumulator), rounded to bf16 once.
#include "l2a_common.cuh"
#include "sm100_prims.cuh"

namespace l2a {

namespace {

constexpr int kBoxBytes = 128 * 128;
constexpr float kLog2e = 1.4426950408889634f;

// ------------------------------------------------------------------------------------------------
// Delta / dgate preprocess.  The grid is one resident wave; the warps take the tokens round-robin, so that at any
// moment the whole grid reads one contiguous stretch of each tensor (a contiguous range per warp, i.e. thousands of
// separate streams, ran at 0.7 of this speed).  A token's Hq*D values are read with 16-byte loads: D/8 lanes per
// head, 32/(D/8) heads per pass, several passes in flight.
__device__ __forceinline__ float dot8(const uint4& x, const uint4& y) {
  const uint32_t a[4] = {x.x, x.y, x.z, x.w}, b[4] = {y.x, y.y, y.z, y.w};
  float acc = 0.f;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    acc = fmaf(__uint_as_float(a[k] << 16), __uint_as_float(b[k] << 16), acc);
    acc = fmaf(__uint_as_float(a[k] & 0xffff0000u), __uint_as_float(b[k] & 0xffff0000u), acc);
  }
  return acc;
}

template <int D>
__global__ void __launch_bounds__(256) bwd_delta_kernel(const bf16* __restrict__ dO, const bf16* __restrict__ dO_loc,
                                                        const bf16* __restrict__ S,
                                                        const bf16* __restrict__ A_c,
                                                        const uint8_t* __restrict__ d_mask,
                                                        const int32_t* __restrict__ prefix, float* __restrict__ delta_loc,
                                                        float* __restrict__ delta_glb, float* __restrict__ dgate, int B,
                                                        int L, int Hq, int a_by_row, int64_t do_bs, int64_t do_ts,
                                                        const float* __restrict__ lse_loc,
                                                        const float* __restrict__ lse_glb, float* __restrict__ lse_eff) {
  constexpr int kLanesPerHead = D / 8;                 // 16-byte chunks per head row
  constexpr int kHeadsPerPass = 32 / kLanesPerHead;
  const int lane = threadIdx.x & 31;
  const int64_t n_tokens = (int64_t)B * L;
  const int64_t n_warps = (int64_t)gridDim.x * (blockDim.x >> 5);
  const int64_t gw = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const bool split = dO_loc != dO;                     // separate gradient for the local output
  const int sub = lane / kLanesPerHead;                // head inside the pass
  const int n_pass = (Hq + kHeadsPerPass - 1) / kHeadsPerPass;
  for (int64_t token = gw; token < n_tokens; token += n_warps) {
    const int b = (int)(token / L), t = (int)(token % L);
    const bool routed = d_mask != nullptr && d_mask[token] != 0;     // NULL: the global part is skipped
    const int c = routed ? prefix[(int64_t)b * (L + 1) + t] : 0;
    // a_by_row: the global output was computed for every token and A is indexed by row (forced-global iterations)
    const bool with_a = routed || a_by_row;
    const int64_t row = token * Hq * D;                          // S: dense
    const int64_t orow = b * do_bs + t * do_ts;                  // dO, dO_loc: the strides of O
    const int64_t crow = ((int64_t)b * L + (a_by_row ? t : c)) * Hq * D;
    const uint4* po = reinterpret_cast<const uint4*>(dO + orow) + lane;
    const uint4* pl = reinterpret_cast<const uint4*>(dO_loc + orow) + lane;
    const uint4* ps = reinterpret_cast<const uint4*>(S + row) + lane;
    const uint4* pa = reinterpret_cast<const uint4*>(A_c + crow) + lane;
    float gate = 0.f;
    // shared-window statistics: the two log-sum-exps of head (32 j + lane), fetched ahead of the passes that need them
    float pre_loc[2] = {0.f, 0.f}, pre_glb[2] = {0.f, 0.f};
    if (lse_eff != nullptr) {
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int h = 32 * j + lane;
        if (h < Hq) {
          pre_loc[j] = __ldg(&lse_loc[((int64_t)b * Hq + h) * L + t]);
          if (routed) pre_glb[j] = __ldg(&lse_glb[((int64_t)b * Hq + h) * L + c]);
        }
      }
    }
#pragma unroll 4
    for (int p = 0; p < n_pass; ++p) {
      const int h = p * kHeadsPerPass + sub;
      float dl = 0.f, dg = 0.f;
      if (h < Hq) {
        const uint4 o = __ldg(po + p * 32);
        if (S != nullptr) dl = dot8(split ? __ldg(pl + p * 32) : o, __ldg(ps + p * 32));   // NULL: local part skipped
        if (with_a) dg = dot8(o, __ldg(pa + p * 32));
      }
#pragma unroll
      for (int off = kLanesPerHead / 2; off > 0; off >>= 1) {
        dl += __shfl_xor_sync(0xffffffffu, dl, off);
        dg += __shfl_xor_sync(0xffffffffu, dg, off);
      }
      // (every lane takes part in the shuffles; heads beyond 64 fall back to loads in place)
      float pre_l = __shfl_sync(0xffffffffu, (h & 32) ? pre_loc[1] : pre_loc[0], h & 31);
      float pre_g = __shfl_sync(0xffffffffu, (h & 32) ? pre_glb[1] : pre_glb[0], h & 31);
      if (h < Hq && (lane % kLanesPerHead) == 0) {
        const int64_t it = ((int64_t)b * Hq + h) * L + t, ic = ((int64_t)b * Hq + h) * L + c;
        if (lse_eff != nullptr && h >= 64) {
          pre_l = lse_loc[it];
          pre_g = routed ? lse_glb[ic] : 0.f;
        }
        float dl_out = dl;
        if (lse_eff != nullptr) {
          // Shared-window backward.  Inside the window of a routed row P_glb = beta * P_loc with
          // beta = exp(lse_loc - lse_glb), and dP is the same product dO V^T for both modules, so the two
          // contributions add up to P' (dP - Delta') with P' = (1 + beta) P_loc and
          // Delta' = (Delta_loc + beta * Delta_glb) / (1 + beta): the local items carry them with these statistics.
          float le = pre_l;
          if (routed) {
            const float beta = __expf(le - pre_g);
            dl_out = (dl + beta * dg) / (1.0f + beta);
            le -= log1pf(beta);
          }
          lse_eff[it] = le;
        }
        if (S != nullptr) delta_loc[it] = dl_out;
        if (routed) delta_glb[ic] = dg;
        gate += dg;
      }
    }
    if (dgate != nullptr) {
#pragma unroll
      for (int off = 16; off >= kLanesPerHead; off >>= 1) gate += __shfl_xor_sync(0xffffffffu, gate, off);
      if (lane == 0) dgate[token] = with_a ? gate : 0.f;
    }
  }
}

// lse by row -> lse by compact row (forced-global iterations store the global log-sum-exp for every row)
__global__ void __launch_bounds__(256) compact_stat_kernel(const float* __restrict__ by_row, float* __restrict__ by_c,
                                                           const int32_t* __restrict__ q_idx,
                                                           const int32_t* __restrict__ n_routed, int L, int Hq) {
  const int b = blockIdx.z, h = blockIdx.y;
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c < n_routed[b]) {
    const int64_t base = ((int64_t)b * Hq + h) * L;
    by_c[base + c] = by_row[base + q_idx[(int64_t)b * L + c]];
  }
}

// ------------------------------------------------------------------------------------------------
struct BwdArgs {
  int B, Lq, Lk, Hq, Hkv, D;
  int window, q_pos_offset;
  float scale, scale_log2;
  int skip_local, skip_global;   // gradients of one module only (the other module has its own Q/K/V)
  int kb_begin, kb_count;        // key blocks [kb_begin, kb_begin + kb_count) of every KV head
  RowStrides dq_st, dk_st, dv_st;   // strides of the gradient tensors in elements
  float* dq_acc_loc;             // fp32 dQ accumulators (layout: see bwd_kernel), by row tile
  float* dq_acc_glb;             //                 and by compact tile; NULL when that module is skipped
  int vis_shift;                 // global items see the keys 0 .. pos - vis_shift: 0, or W + 1 when the window's share of
                                 // the global gradient is carried by the local items (shared-window backward)
  const int32_t* q_idx;
  const int32_t* n_routed;
  const int32_t* prefix;
  const int32_t* seq_bounds;   // packed sequences (B == 1): per token {first token of its sequence, one past the last}
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
// Thread roles of the tensor-core kernel below:
//   warps 0-15 : compute.  Warp w owns TMEM lanes 32*(w%4)..+31 (its thread's key, or query row of dQ) and the
//                32 score columns of quarter w/4, so that 16 warps hide each other's TMEM and MUFU latency.
//   warp 16    : TMA producer          warp 17 : tcgen05 MMA issuer, TMEM owner
//   warp 18    : stages the row statistics of each query tile          warp 19 : idle
//   warps 20-27: read every dQ(i) tile out of TMEM (one lane group and one half of the columns each) and add it into the
//                fp32 accumulators: the reductions leave an SM at about 32 bytes per clock, and a warp that issues them
//                stalls that long, so they are kept off the warps whose progress the tensor pipe waits for.  A read-out
//                warp takes its whole share (64 values per thread) into registers and releases the TMEM columns before
//                its first reduction.
// Registers: 896 threads start with 72 each (64512 in all, which is also all that setmaxnreg can redistribute: an
// increase is served from what the CTA's own warps released); the service warpgroup goes down to 40, the read-out
// warpgroups stay at 72, the compute warpgroups go up to 80 -- which they fit because scores and dP^T leave TMEM sixteen
// columns at a time.
constexpr int kComputeWarps = 16;
constexpr int kDkvThreads = 28 * 32;   // 896

__device__ __forceinline__ float bf16lo_to_f32(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t packed) { return __uint_as_float(packed & 0xffff0000u); }

struct ItemPlan {
  int loc_t0, loc_nt;   // first local query tile, number of local tiles
  int glb_t0, glb_nt;   // first compact tile, number of compact tiles
  int per_head;         // loc_nt + glb_nt
  int total;            // per_head * G
};

__device__ __forceinline__ ItemPlan make_plan(const BwdArgs& a, int b, int k0, int span = kTileN) {
  ItemPlan p;
  // packed sequences: no row at or after the end of the sequence that holds the block's last key sees any of its keys
  int row_end = a.Lq;
  if (a.seq_bounds != nullptr) {
    const int k_last = min(k0 + span, a.Lk) - 1;
    row_end = max(0, min(a.Lq, a.seq_bounds[2 * k_last + 1]));
  }
  // local: rows t with position in [k0, k0 + span - 1 + W]
  int tmin = k0 - a.q_pos_offset;
  const long long tmax_ll = (long long)k0 + span - 1 + a.window - a.q_pos_offset;
  int tmax = tmax_ll > row_end - 1 ? row_end - 1 : (int)tmax_ll;
  if (tmin < 0) tmin = 0;
  if (tmax < tmin || a.skip_local) { p.loc_t0 = 0; p.loc_nt = 0; }
  else { p.loc_t0 = tmin / kTileM; p.loc_nt = tmax / kTileM - p.loc_t0 + 1; }
  // global: compact rows whose last visible key (position - vis_shift) is >= k0
  const int n_c = a.skip_global ? 0 : a.n_routed[b];
  long long tmin_g = (long long)k0 - a.q_pos_offset + a.vis_shift;
  if (tmin_g < 0) tmin_g = 0;
  if (tmin_g > row_end - 1 || n_c == 0) { p.glb_t0 = 0; p.glb_nt = 0; }
  else {
    const int c_min = a.prefix[(int64_t)b * (a.Lq + 1) + (int)tmin_g];
    const int c_end = row_end < a.Lq ? min(n_c, a.prefix[(int64_t)b * (a.Lq + 1) + row_end]) : n_c;
    if (c_min >= c_end) { p.glb_t0 = 0; p.glb_nt = 0; }
    else { p.glb_t0 = c_min / kTileM; p.glb_nt = (c_end - 1) / kTileM - p.glb_t0 + 1; }
  }
  p.per_head = p.loc_nt + p.glb_nt;
  p.total = p.per_head * (a.Hq / a.Hkv);
  return p;
}

// Walks the items of a CTA in order without divisions: (head, local/compact, tile).
struct ItemCursor {
  int h, r, per_head, loc_nt, loc_t0, glb_t0;
  __device__ __forceinline__ ItemCursor(const ItemPlan& p, int h0)
      : h(h0), r(0), per_head(p.per_head), loc_nt(p.loc_nt), loc_t0(p.loc_t0), glb_t0(p.glb_t0) {}
  __device__ __forceinline__ int glb() const { return r >= loc_nt; }
  __device__ __forceinline__ int tile() const { return r < loc_nt ? loc_t0 + r : glb_t0 + (r - loc_nt); }
  __device__ __forceinline__ void next() { if (++r == per_head) { r = 0; ++h; } }
};

// ================================================================================================
// Five-GEMM backward kernel: the key/value-stationary kernel above plus the fifth GEMM, dQ(i) = dS(i) K, so that
// S and dP are computed once per tile pair.  dQ(i) is a fresh 128 x D accumulator per item; the read-out warps take
// it out (lane = query row) and add it into an fp32 accumulator in global memory whose layout is private to this
// file: per (batch, head, 128-row tile) one block of 128 x D floats ordered [warp 16][piece D/16][lane 32][4], so
// that every red.global.add.v4.f32 of a warp covers 512 contiguous bytes.  Local items add into the accumulator
// indexed by row tile, global items into the one indexed by compact tile; dq_merge_kernel forms the bf16 dQ.
// All key blocks meet in those accumulators in no fixed order: dQ is not bit-reproducible from run to run
// (dK, dV are).
//   TMEM: dV [0,D) | dK [D,2D) | T [256,384): S^T(i), then P^T(i) (bf16, quarter-local) | U [384,512): dP^T(i),
//         then dQ(i).
//   Shared memory: K, V resident; Q and dO in two-stage rings; dS(i) (bf16, [key][query], swizzled like a TMA
//   tile) -- the A operand of both dK += dS^T Q (read K-major) and dQ = dS K (read MN-major).
//   MMA order per item i:  dV(i) | S^T(i+1) | dQ(i) | dK(i) | dP^T(i+1).  S^T(i+1) does not depend on dS(i), so it is
//   issued ahead of the wait for it: the compute warps find the next scores ready when they are done with dS(i).
//   Two loops run through the order: T: S^T -> P -> dV -> S^T and U: dP^T -> dS -> dQ -> read-out -> dP^T; dK(i) keeps the
//   pipe busy while the read-out warps take dQ(i) out of TMEM, which frees U well before their reductions are issued.

// The reductions of one read-out warp: piece I of its 32 x D/2 share (4 columns each) goes to a byte offset from the
// warp's base address that is a compile-time constant, so that all of them share one address register pair.
template <int kBytes>
__device__ __forceinline__ void red_add_v4(float* base, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("red.global.add.v4.f32 [%0+%5], {%1, %2, %3, %4};" ::"l"(base), "f"(__uint_as_float(a)),
               "f"(__uint_as_float(b)), "f"(__uint_as_float(c)), "f"(__uint_as_float(d)), "n"(kBytes)
               : "memory");
}
// Least distance between two reductions of a read-out warp, in SM clocks (polled: a sleep is too coarse).  Sixteen
// reductions then take about 1800 clocks of an item's 4000 or more; 96 to 128 measure the same, 64 and 160 are slower.
constexpr int kRedSpacingClk = 112;
template <int D, int I>
struct ReadOutReds {
  static constexpr int kCols = D / 4;                 // columns per quarter of the accumulator layout
  static constexpr int kCol = 4 * I;                  // relative to the warp's first column
  static constexpr int kOff = ((kCol / kCols) * 4 * (8 * D) + ((kCol % kCols) / 4) * 128) * 4;
  __device__ __forceinline__ static void run(float* base, const uint32_t (&v)[D / 64][32]) {
    // spaced out: reductions issued back to back fill the queue of the memory pipe, and the compute warps' shared-memory
    // loads and stores (row statistics, dS) wait behind them; the read-out warps have most of an item's time to spare
    { const long long t0 = clock64(); while (clock64() - t0 < kRedSpacingClk) { } }
    red_add_v4<kOff>(base, v[I / 8][4 * (I % 8)], v[I / 8][4 * (I % 8) + 1], v[I / 8][4 * (I % 8) + 2],
                     v[I / 8][4 * (I % 8) + 3]);
    ReadOutReds<D, I + 1>::run(base, v);
  }
};
template <int D>
struct ReadOutReds<D, D / 8> {
  __device__ __forceinline__ static void run(float*, const uint32_t (&)[D / 64][32]) {}
};

template <int D>
struct BwdSmem {
  static constexpr int kTileBytes = 128 * D * 2;
  static constexpr int kKOff = 0;
  static constexpr int kVOff = kTileBytes;
  static constexpr int kQOff = 2 * kTileBytes;                 // 2 stages
  static constexpr int kDoOff = kQOff + 2 * kTileBytes;        // 2 stages
  static constexpr int kDsOff = kDoOff + 2 * kTileBytes;       // dS: 128 keys x 128 queries bf16
  static constexpr int kStatOff = kDsOff + 128 * 128 * 2;
  static constexpr int kStatSlot = (2 * 128 + 8) * 4;
  static constexpr int kBarOff = kStatOff + 2 * kStatSlot;
  static constexpr int kTotal = kBarOff + 256;
};
struct BwdBarriers {
  uint64_t kv_full;
  uint64_t q_full[2], q_empty[2];
  uint64_t do_full[2], do_empty[2];
  uint64_t st_full[2], st_empty[2];
  uint64_t s_full, dp_full, p_full, ds_full, ds_free, dq_full, u_free, final_bar;
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(BwdBarriers) <= 256, "barrier block");

template <int D>
__global__ void __launch_bounds__(kDkvThreads, 1)
bwd_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapDO,
               const __grid_constant__ CUtensorMap mapQc, const __grid_constant__ CUtensorMap mapDOc,
               const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV, const BwdArgs a) {
  using SM = BwdSmem<D>;
  constexpr int kKSteps = D / 16;
  // key blocks ascending (most work first) inside one KV head; KV heads outermost so that the CTAs
  // running together share the same query tiles in L2
  const int j = a.kb_begin + blockIdx.x % a.kb_count;
  const int rest = blockIdx.x / a.kb_count;
  const int b = rest % a.B;
  const int g = rest / a.B;
  const int G = a.Hq / a.Hkv;
  const int k0 = j * kTileN;
  const ItemPlan plan = make_plan(a, b, k0);
  const int n_c = a.skip_global ? 0 : a.n_routed[b];   // the routing arrays may be NULL when the global part is skipped

  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* sK = smem + SM::kKOff;
  uint8_t* sV = smem + SM::kVOff;
  uint8_t* sQ = smem + SM::kQOff;
  uint8_t* sDO = smem + SM::kDoOff;
  BwdBarriers* bar = reinterpret_cast<BwdBarriers*>(smem + SM::kBarOff);
  uint8_t* sDS = smem + SM::kDsOff;          // dS (bf16, [key][query])
  volatile int* abort_flag = &bar->abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if ((smem_u32(smem) & 1023u) != 0) {   // the swizzled tiles need a 1024-byte aligned base: refuse to run otherwise
    if (tid == 0) atomicExch(a.status, 2);
    return;
  }
  if (plan.total == 0) {
    // no query can see these keys: their gradients are zero
    for (int i = tid; i < kTileN * (D / 8); i += blockDim.x) {
      const int kr = i / (D / 8), c8 = i % (D / 8);
      if (k0 + kr < a.Lk) {
        const int64_t o = (int64_t)g * D + c8 * 8;
        *reinterpret_cast<uint4*>(a.dK + b * a.dk_st.b + (k0 + kr) * a.dk_st.t + o) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(a.dV + b * a.dv_st.b + (k0 + kr) * a.dv_st.t + o) = make_uint4(0, 0, 0, 0);
      }
    }
    return;
  }

  if (tid == 0) {
    mbar_init(&bar->kv_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bar->q_full[s], 1); mbar_init(&bar->q_empty[s], 1);
      mbar_init(&bar->do_full[s], 1); mbar_init(&bar->do_empty[s], 1);
      mbar_init(&bar->st_full[s], 32); mbar_init(&bar->st_empty[s], kComputeWarps * 32);
    }
    mbar_init(&bar->s_full, 1);
    mbar_init(&bar->dp_full, 1);
    mbar_init(&bar->p_full, kComputeWarps * 32);     // P^T(i) is in TMEM
    mbar_init(&bar->ds_full, kComputeWarps * 32);    // dS(i) is in shared memory and dP^T(i) has been read
    mbar_init(&bar->ds_free, 1);                     // dQ(i) and dK(i) have consumed dS(i)
    mbar_init(&bar->dq_full, 1);                     // dQ(i) is in TMEM
    mbar_init(&bar->u_free, 8 * 32);     // dQ(i) has been read out: the columns may take dP^T(i+1)
    mbar_init(&bar->final_bar, 1);
    bar->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 17) { tmem_alloc(&bar->tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bar->tmem_base;
  if (tmem != 0) {
    // all 512 columns were requested, so the allocation must start at column 0; the MMA warp relies on it to
    // keep its TMEM operand addresses compile-time constants
    __syncthreads();
    if (warp == 17) tmem_dealloc(tmem, 512);
    if (tid == 0) atomicExch(a.status, 3);
    return;
  }

  // register shares by warpgroup: every warp of a warpgroup executes the same setmaxnreg at the top of its role
  if (warp >= 20) {
    // ------------------------------------------------------------------ dQ read-out: TMEM -> fp32 accumulators
    setmaxnreg_dec<72>();
    // lane == query row of the item's tile; this warp owns the 32 rows of its lane group and one half of the D columns,
    // read in one go: each 32 x 4 piece is then one 512-byte reduction (accumulator layout: see above)
    const int grp = warp & 3, half = (warp - 20) >> 2;
    const uint32_t lane_base = static_cast<uint32_t>(grp * 32) << 16;
    const int n_tiles = (a.Lq + kTileM - 1) / kTileM;
    constexpr int kChunks = D / 32;     // 32-column TMEM loads of the whole tile; this warp takes half of them
    ItemCursor cur(plan, g * G);
    for (int i = 0; i < plan.total; ++i) {
      const int h = cur.h, glb = cur.glb(), tile = cur.tile();
      cur.next();
      float* acc = glb ? a.dq_acc_glb : a.dq_acc_loc;
      const bool item_ok = dbg_in_range(tile >= 0 && tile < n_tiles && h >= 0 && h < a.Hq && acc != nullptr, a.status);
      acc += (((int64_t)b * a.Hq + h) * n_tiles + tile) * (int64_t)(kTileM * D) + lane * 4;
      if (!__all_sync(0xffffffffu, mbar_wait(&bar->dq_full, i & 1, abort_flag))) break;
      tc_fence_after();
      // the warp's whole share (32 rows x D/2 columns) goes to registers first, so that the region is released before
      // the first reduction is issued: the reductions leave the SM at about 32 bytes per clock and must not hold up
      // dP^T(i+1)
      uint32_t v[kChunks / 2][32];
#pragma unroll
      for (int cc = 0; cc < kChunks / 2; ++cc) tmem_ld32(tmem + lane_base + 384 + (half * (kChunks / 2) + cc) * 32, v[cc]);
      tmem_ld_wait();
      tc_fence_before();
      mbar_arrive(&bar->u_free);           // everything is in registers: dP^T(i+1) may overwrite the columns
      if (item_ok) {
        // this warp's columns start at (D / 2) * half, i.e. at quarter 2 * half of the accumulator layout; every further
        // offset is a compile-time constant, so that the sixteen reductions share one address register pair
        float* base = acc + ((2 * half) * 4 + grp) * (8 * D);
        ReadOutReds<D, 0>::run(base, v);
      }
    }
  } else if (warp == 19) {
    setmaxnreg_dec<40>();     // idle
  } else if (warp == 16) {
    // ------------------------------------------------------------------ TMA producer
    setmaxnreg_dec<40>();
    if (lane == 0) {
      tma_prefetch_desc(&mapQ); tma_prefetch_desc(&mapDO); tma_prefetch_desc(&mapQc); tma_prefetch_desc(&mapDOc);
      mbar_expect_tx(&bar->kv_full, 2 * SM::kTileBytes);
      tma_load_4d(sK, &mapK, &bar->kv_full, 0, k0, g * (D / 64), b);
      tma_load_4d(sV, &mapV, &bar->kv_full, 0, k0, g * (D / 64), b);
      ItemCursor cur(plan, g * G);
      for (int i = 0; i < plan.total; ++i) {
        const int glb = cur.glb(), row0 = cur.tile() * kTileM, hc = cur.h * (D / 64);
        cur.next();
        const int st = i & 1;
        const uint32_t ph = ((i >> 1) & 1) ^ 1;
        if (!mbar_wait(&bar->q_empty[st], ph, abort_flag)) break;
        mbar_expect_tx(&bar->q_full[st], SM::kTileBytes);
        tma_load_4d(sQ + st * SM::kTileBytes, glb ? &mapQc : &mapQ, &bar->q_full[st], 0, row0, hc, b);
        if (!mbar_wait(&bar->do_empty[st], ph, abort_flag)) break;
        mbar_expect_tx(&bar->do_full[st], SM::kTileBytes);
        tma_load_4d(sDO + st * SM::kTileBytes, glb ? &mapDOc : &mapDO, &bar->do_full[st], 0, row0, hc, b);
      }
    }
    __syncwarp();
  } else if (warp == 18) {
    // ------------------------------------------------------------------ row statistics of each item
    setmaxnreg_dec<40>();
    // lse * log2(e) and Delta of the item's 128 query rows, plus per-quarter mask flags, go to shared memory.
    // The global loads of item i+1 are issued before waiting for its slot, so their latency is hidden.
    float r_lse[4], r_delta[4];
    int r_pos[4], r_lo[4], r_glb = 0, r_row0 = 0, r_h = 0;   // r_lo: first token of the row's sequence (packed batches)
    ItemCursor cur(plan, g * G);
    auto load_item = [&]() {
      const int h = cur.h, glb = cur.glb(), row0 = cur.tile() * kTileM;
      cur.next();
      const int n_rows = glb ? n_c : a.Lq;
      const float* lse = glb ? a.lse_glb : a.lse_loc;
      const float* dl = glb ? a.delta_glb : a.delta_loc;
      r_glb = glb;
      r_row0 = row0;
      r_h = h;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int row = row0 + q * 32 + lane;
        const bool valid = row < n_rows;
        const int64_t si = ((int64_t)b * a.Hq + h) * a.Lq + (valid ? row : 0);
        r_lse[q] = valid ? __ldg(&lse[si]) * kLog2e : 0.f;
        r_delta[q] = valid ? __ldg(&dl[si]) : 0.f;
        const int token = valid ? (glb ? __ldg(&a.q_idx[(int64_t)b * a.Lq + row]) : row) : 0;
        r_pos[q] = valid ? token - (glb ? a.vis_shift : 0) + a.q_pos_offset : -1;
        r_lo[q] = (valid && a.seq_bounds != nullptr) ? __ldg(&a.seq_bounds[2 * token]) : -0x40000000;
      }
    };
    load_item();
    for (int i = 0; i < plan.total; ++i) {
      const int s = i & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(&bar->st_empty[s], ((i >> 1) & 1) ^ 1, abort_flag))) break;
      float* st_lse = reinterpret_cast<float*>(smem + SM::kStatOff + s * SM::kStatSlot);
      float* st_delta = st_lse + 128;
      int* st_flags = reinterpret_cast<int*>(st_delta + 128);
      const int w_eff = r_glb ? 0x3fffffff : a.window;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int col = q * 32 + lane;
        st_lse[col] = -r_lse[q];       // negated, like Delta: P = exp2(scale * s + (-lse)) is one fused multiply-add
        st_delta[col] = -r_delta[q];   // negated: dS = P * (dP + (-Delta)) with packed f32x2 arithmetic
        // quarter q needs the element mask unless every (key, query) pair of it is visible
        const bool lane_ok = r_pos[q] >= 0 && (k0 + kTileN - 1 <= r_pos[q]) && (k0 >= max(r_pos[q] - w_eff, r_lo[q]));
        const bool interior = __all_sync(0xffffffffu, lane_ok);
        if (lane == 0) st_flags[q] = interior ? 0 : 1;
      }
      if (lane == 0) { st_flags[4] = r_glb; st_flags[5] = r_row0; st_flags[6] = r_h; }
      __syncwarp();
      mbar_arrive(&bar->st_full[s]);
      if (i + 1 < plan.total) load_item();
    }
  } else if (warp == 17) {
    // ------------------------------------------------------------------ MMA issuer
    // (whole warp runs the loop; only the tcgen05 instructions are predicated on lane 0)
    setmaxnreg_dec<40>();
    {
      const uint32_t leader = (lane == 0);
      constexpr uint32_t tmem = 0;   // checked above: TMEM operand addresses are immediates in this loop
      constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0);
      constexpr uint32_t idesc_acc = idesc_bf16_f32(128, D, 0, 1);
      constexpr uint32_t idesc_dq = idesc_bf16_f32(128, D, 1, 1);     // A = dS read MN-major, B = K read MN-major
      constexpr uint32_t kStageStep = SM::kTileBytes >> 4;
      const uint64_t dk = smem_desc_sw128(smem_u32(sK), 16, 1024), dv = smem_desc_sw128(smem_u32(sV), 16, 1024);
      const uint64_t dkm = smem_desc_sw128(smem_u32(sK), kBoxBytes, 1024);            // K as MN-major B of dQ
      const uint64_t dsm = smem_desc_sw128(smem_u32(sDS), kBoxBytes, 1024);           // dS as MN-major A of dQ
      const uint64_t dsk = smem_desc_sw128(smem_u32(sDS), 16, 1024);                  // dS^T as K-major A of dK
      const uint64_t dq_base = smem_desc_sw128(smem_u32(sQ), 16, 1024);
      const uint64_t ddo_base = smem_desc_sw128(smem_u32(sDO), 16, 1024);
      const uint64_t dqm_base = smem_desc_sw128(smem_u32(sQ), kBoxBytes, 1024);      // Q / dO as MN-major B
      const uint64_t ddom_base = smem_desc_sw128(smem_u32(sDO), kBoxBytes, 1024);
      auto issue_S = [&](int qs) {    // S^T = K Q^T into the T columns
        const uint64_t qd = dq_base + qs * kStageStep;
#pragma unroll
        for (int kk = 0; kk < kKSteps; ++kk) {
          const uint32_t c = ((kk >> 2) * kBoxBytes + (kk & 3) * 32) >> 4;
          mma_ss(tmem + 256, dk + c, qd + c, idesc_s, kk > 0, leader);
        }
        tc_commit(&bar->s_full, leader);
      };
      auto issue_dP = [&](int ds) {   // dP^T = V dO^T into the U columns
        const uint64_t dod = ddo_base + ds * kStageStep;
#pragma unroll
        for (int kk = 0; kk < kKSteps; ++kk) {
          const uint32_t c = ((kk >> 2) * kBoxBytes + (kk & 3) * 32) >> 4;
          mma_ss(tmem + 384, dv + c, dod + c, idesc_s, kk > 0, leader);
        }
        tc_commit(&bar->dp_full, leader);
      };
      auto issue_dQ = [&]() {         // dQ(i) = dS K into the U columns (a fresh accumulator for every item)
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          mma_ss(tmem + 384, dsm + ((kk * 2048) >> 4), dkm + ((kk * 2048) >> 4), idesc_dq, kk > 0, leader);
        tc_commit(&bar->dq_full, leader);
      };
      auto issue_dV = [&](int ds, bool first) {   // dV += P^T dO, P^T from the T columns
        const uint64_t dod = ddom_base + ds * kStageStep;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          mma_ts(tmem, tmem + 256 + (kk >> 1) * 32 + (kk & 1) * 8, dod + ((kk * 2048) >> 4), idesc_acc,
                 (kk > 0 || !first) ? 1u : 0u, leader);
        tc_commit(&bar->do_empty[ds], leader);
      };
      auto issue_dK = [&](int qs, bool first) {   // dK += dS^T Q, dS^T from shared memory
        const uint64_t qd = dqm_base + qs * kStageStep;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t c = ((kk >> 2) * kBoxBytes + (kk & 3) * 32) >> 4;
          mma_ss(tmem + D, dsk + c, qd + ((kk * 2048) >> 4), idesc_acc, (kk > 0 || !first) ? 1u : 0u, leader);
        }
        tc_commit(&bar->q_empty[qs], leader);
        tc_commit(&bar->ds_free, leader);
      };
      bool ok = mbar_spin_warp(&bar->kv_full, 0, abort_flag) && mbar_spin_warp(&bar->q_full[0], 0, abort_flag) &&
                mbar_spin_warp(&bar->do_full[0], 0, abort_flag);
      if (ok) {
        tc_fence_after();
        issue_S(0);
        issue_dP(0);
      }
      for (int i = 0; ok && i < plan.total; ++i) {
        const bool more = i + 1 < plan.total;
        if (!mbar_spin_warp(&bar->p_full, i & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        issue_dV(i & 1, i == 0);
        if (more) {
          // S^T(i+1) overwrites P^T(i): dV(i) precedes it in issue order.  It does not depend on dS(i), so it goes
          // ahead of that wait: the compute warps find the next scores ready when they are done with dS(i)
          if (!mbar_spin_warp(&bar->q_full[(i + 1) & 1], ((i + 1) >> 1) & 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
          issue_S((i + 1) & 1);
        }
        if (!mbar_spin_warp(&bar->ds_full, i & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        issue_dQ();
        issue_dK(i & 1, i == 0);       // keeps the pipe busy while dQ(i) is read out
        if (more) {
          const int sn = (i + 1) & 1;
          const uint32_t phn = ((i + 1) >> 1) & 1;
          // dP^T(i+1) overwrites dQ(i): wait for its read-out
          if (!mbar_spin_warp(&bar->u_free, i & 1, abort_flag) ||
              !mbar_spin_warp(&bar->do_full[sn], phn, abort_flag)) { ok = false; break; }
          tc_fence_after();
          issue_dP(sn);
        }
      }
      if (ok) tc_commit(&bar->final_bar, leader);
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ P^T, dS and epilogue
    setmaxnreg_inc<80>();
    const int q = warp >> 2;                           // query-column quarter of this warp
    const int kr = (warp & 3) * 32 + lane;             // key inside the block == TMEM lane
    const int kp = k0 + kr;
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t s_addr = tmem + lane_base + 256 + q * 32;
    const uint32_t dp_addr = tmem + lane_base + 384 + q * 32;
    bool ok = true;
    for (int i = 0; i < plan.total; ++i) {
      const int s = i & 1;
      // this item's row statistics go to registers before the scores are waited for
      if (!__all_sync(0xffffffffu, mbar_wait(&bar->st_full[s], (i >> 1) & 1, abort_flag))) { ok = false; break; }
      const uint32_t st_base = smem_u32(smem + SM::kStatOff + s * SM::kStatSlot);
      const int* st_flags = reinterpret_cast<const int*>(smem + SM::kStatOff + s * SM::kStatSlot) + 2 * 128;
      float st[32];
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const float4 v = lds128(st_base + (q * 32 + c * 4) * 4);
        st[4 * c] = v.x; st[4 * c + 1] = v.y; st[4 * c + 2] = v.z; st[4 * c + 3] = v.w;
      }
      const bool masked = st_flags[q] != 0;
      const int item_glb = st_flags[4], item_row0 = st_flags[5];
      if (!__all_sync(0xffffffffu, mbar_wait(&bar->s_full, i & 1, abort_flag))) { ok = false; break; }
      tc_fence_after();
      uint32_t pp[16];
      {
        const int w_eff = item_glb ? 0x3fffffff : a.window;
        const int n_rows = item_glb ? n_c : a.Lq;
        const int32_t* qi = a.q_idx + (int64_t)b * a.Lq;
        // the scores come out of TMEM sixteen columns at a time (register budget of the compute warps)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          uint32_t sv[16];
          tmem_ld16(s_addr + hh * 16, sv);
          tmem_ld_wait();
          // the element mask is needed only for the few tiles that straddle the causal diagonal or a window edge:
          // two loop versions, so that the common one has no branches
          if (!masked) {
#pragma unroll
            for (int e8 = 0; e8 < 8; ++e8) {
              const int e = hh * 8 + e8;
              const float2 x = __ffma2_rn(make_float2(__uint_as_float(sv[2 * e8]), __uint_as_float(sv[2 * e8 + 1])),
                                          make_float2(a.scale_log2, a.scale_log2), make_float2(st[2 * e], st[2 * e + 1]));
              pp[e] = pack_bf16(fast_exp2(x.x), fast_exp2(x.y));
            }
          } else {
#pragma unroll
            for (int e16 = 0; e16 < 16; e16 += 2) {
              const int e = hh * 16 + e16;
              int pos[2], lo[2];
#pragma unroll
              for (int u = 0; u < 2; ++u) {
                const int row = item_row0 + q * 32 + e + u;
                const bool valid = row < n_rows;
                const int token = valid ? (item_glb ? __ldg(&qi[row]) : row) : 0;
                pos[u] = valid ? token - (item_glb ? a.vis_shift : 0) + a.q_pos_offset : -1;
                lo[u] = pos[u] - w_eff;
                if (valid && a.seq_bounds != nullptr) lo[u] = max(lo[u], __ldg(&a.seq_bounds[2 * token]));
              }
              float p0 = fast_exp2(fmaf(__uint_as_float(sv[e16]), a.scale_log2, st[e]));
              float p1 = fast_exp2(fmaf(__uint_as_float(sv[e16 + 1]), a.scale_log2, st[e + 1]));
              p0 = (kp <= pos[0] && kp >= lo[0]) ? p0 : 0.f;
              p1 = (kp <= pos[1] && kp >= lo[1]) ? p1 : 0.f;
              pp[e >> 1] = pack_bf16(p0, p1);
            }
          }
        }
      }
      tmem_st16(s_addr, pp);     // P^T over the first half of this quarter's own S^T columns
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(&bar->p_full);
      // -Delta of the same rows, again ahead of the wait; after this the statistics slot may be refilled
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const float4 v = lds128(st_base + (128 + q * 32 + c * 4) * 4);
        st[4 * c] = v.x; st[4 * c + 1] = v.y; st[4 * c + 2] = v.z; st[4 * c + 3] = v.w;
      }
      mbar_arrive(&bar->st_empty[s]);
      if (!__all_sync(0xffffffffu, mbar_wait(&bar->dp_full, i & 1, abort_flag))) { ok = false; break; }
      tc_fence_after();
      uint32_t pd[16];
      // dP^T comes out of TMEM sixteen columns at a time: with the 32 statistics and the 16 packed probabilities live,
      // a 32-column load would not fit the compute warps' 80 registers
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        uint32_t dv[16];
        tmem_ld16(dp_addr + hh * 16, dv);
        tmem_ld_wait();
#pragma unroll
        for (int e8 = 0; e8 < 8; ++e8) {
          const int e = hh * 8 + e8;
          // dS uses the bf16-rounded P, the same value the dV product sees; st[] holds -Delta
          const float2 t = __fadd2_rn(make_float2(__uint_as_float(dv[2 * e8]), __uint_as_float(dv[2 * e8 + 1])),
                                      make_float2(st[2 * e], st[2 * e + 1]));
          const float2 ds = __fmul2_rn(make_float2(bf16lo_to_f32(pp[e]), bf16hi_to_f32(pp[e])), t);
          pd[e] = pack_bf16(ds.x, ds.y);
        }
      }
      // dS goes to shared memory, [key][query] with the 128-byte swizzle of a TMA tile (two boxes of 64 queries); the
      // tile of the previous item must have been consumed by dQ(i-1) and dK(i-1)
      if (i > 0 && !__all_sync(0xffffffffu, mbar_wait(&bar->ds_free, (i - 1) & 1, abort_flag))) { ok = false; break; }
      {
        const uint32_t row = smem_u32(sDS) + (q >> 1) * kBoxBytes + kr * 128;
        const int chunk0 = (q & 1) * 4;
#pragma unroll
        for (int c = 0; c < 4; ++c)
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row + (((chunk0 + c) ^ (kr & 7)) << 4)),
                       "r"(pd[4 * c]), "r"(pd[4 * c + 1]), "r"(pd[4 * c + 2]), "r"(pd[4 * c + 3]) : "memory");
      }
      fence_async_smem();        // the MMA reads the tile through the async proxy
      tc_fence_before();         // orders the dP^T read above before the dQ MMA that overwrites those columns
      mbar_arrive(&bar->ds_full);
    }
    // epilogue: quarters 0,1 store the two column halves of dV, quarters 2,3 those of dK
    if (ok && __all_sync(0xffffffffu, mbar_wait(&bar->final_bar, 0, abort_flag))) {
      tc_fence_after();
      const bool valid = kp < a.Lk;
      const int which = q >> 1, half = q & 1;
      const RowStrides st = which == 0 ? a.dv_st : a.dk_st;
      const int64_t o = b * st.b + (valid ? kp : 0) * st.t + (int64_t)g * D + half * (D / 2);
      bf16* dst = (which == 0 ? a.dV : a.dK) + o;
      const float mul = which == 0 ? 1.0f : a.scale;
#pragma unroll
      for (int c = 0; c < D / 64; ++c) {
        uint32_t v[32];
        tmem_ld32(tmem + lane_base + which * D + half * (D / 2) + c * 32, v);
        tmem_ld_wait();
        if (valid) {
          uint4* d4 = reinterpret_cast<uint4*>(dst + c * 32);
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            float f[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[8 * x + e]) * mul;
            d4[x] = make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]),
                               pack_bf16(f[6], f[7]));
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
  if (warp == 17) tmem_dealloc(tmem, 512);
}

// Zeroes the fp32 dQ accumulators: every row tile of the local one, the compact tiles below n_routed of the global one.
__global__ void __launch_bounds__(256) dq_zero_kernel(float* __restrict__ acc_loc, float* __restrict__ acc_glb,
                                                      const int32_t* __restrict__ n_routed, int B, int Hq, int n_tiles,
                                                      int tile_floats) {
  const int per = B * Hq * n_tiles;
  for (int item = blockIdx.x; item < 2 * per; item += gridDim.x) {
    const int which = item >= per, rem = which ? item - per : item;
    float* base = which ? acc_glb : acc_loc;
    if (base == nullptr) continue;
    if (which && (rem % n_tiles) * kTileM >= n_routed[rem / (n_tiles * Hq)]) continue;
    float4* p = reinterpret_cast<float4*>(base + (int64_t)rem * tile_floats);
    for (int k = threadIdx.x; k < tile_floats / 4; k += blockDim.x) p[k] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
}

// fp32 dQ accumulators -> bf16 dQ: dQ_t = scale * (local(t) + d_t * global(prefix[t])), for the row tiles
// [tile_begin, tile_begin + tile_count).  One CTA per (batch, row tile, head); the accumulator blocks are read in their own order (512 contiguous bytes per warp), the bf16 rows leave
// through shared memory as whole 2 D-byte segments.
template <int D>
__global__ void __launch_bounds__(256) dq_merge_kernel(const float* __restrict__ acc_loc, const float* __restrict__ acc_glb,
                                                       const uint8_t* __restrict__ d_mask,
                                                       const int32_t* __restrict__ prefix, bf16* __restrict__ dQ, int B,
                                                       int L, int Hq, float scale, int64_t bs, int64_t ts,
                                                       int tile_begin, int tile_count, int* status) {
  constexpr int kChunks = D / 8;             // 16-byte chunks per bf16 row
  constexpr int kRowBytes = D * 2 + 16;      // padded: conflict-free 16-byte accesses down a column
  __shared__ __align__(16) uint8_t tile_s[kTileM * kRowBytes];
  const int n_tiles = (L + kTileM - 1) / kTileM;
  const int h = blockIdx.x % Hq;
  const int tile = tile_begin + (blockIdx.x / Hq) % tile_count;
  const int b = blockIdx.x / (Hq * tile_count);
  const int64_t tile_floats = kTileM * D;
  const float* loc = acc_loc ? acc_loc + (((int64_t)b * Hq + h) * n_tiles + tile) * tile_floats : nullptr;
  for (int idx = threadIdx.x; idx < kTileM * kChunks; idx += blockDim.x) {
    const int lane = idx & 31, rq = (idx >> 5) & 3, k = idx >> 7;
    const int r = rq * 32 + lane, t = tile * kTileM + r;
    if (t >= L) continue;
    const int d0 = 8 * k, q = d0 / (D / 4), c = (d0 % (D / 4)) / 4;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f), y = x;
    if (loc) {
      const float4* p = reinterpret_cast<const float4*>(loc + (q * 4 + rq) * (8 * D) + c * 128 + lane * 4);
      x = __ldg(p); y = __ldg(p + 32);
    }
    if (acc_glb && d_mask[(int64_t)b * L + t]) {
      const int cr = prefix[(int64_t)b * (L + 1) + t];
      if (!dbg_in_range(cr >= 0 && cr < n_tiles * kTileM, status)) continue;
      const float4* p = reinterpret_cast<const float4*>(
          acc_glb + (((int64_t)b * Hq + h) * n_tiles + (cr >> 7)) * tile_floats + (q * 4 + ((cr & 127) >> 5)) * (8 * D) +
          c * 128 + (cr & 31) * 4);
      const float4 gx = __ldg(p), gy = __ldg(p + 32);
      x.x += gx.x; x.y += gx.y; x.z += gx.z; x.w += gx.w;
      y.x += gy.x; y.y += gy.y; y.z += gy.z; y.w += gy.w;
    }
    *reinterpret_cast<uint4*>(tile_s + r * kRowBytes + k * 16) =
        make_uint4(pack_bf16(x.x * scale, x.y * scale), pack_bf16(x.z * scale, x.w * scale),
                   pack_bf16(y.x * scale, y.y * scale), pack_bf16(y.z * scale, y.w * scale));
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < kTileM * kChunks; idx += blockDim.x) {
    const int r = idx / kChunks, k = idx % kChunks, t = tile * kTileM + r;
    if (t < L)
      *reinterpret_cast<uint4*>(dQ + b * bs + t * ts + (int64_t)h * D + k * 8) =
          *reinterpret_cast<const uint4*>(tile_s + r * kRowBytes + k * 16);
  }
}

}  // namespace
int delta_ctas_per_sm(int D) {
  int per_sm = 0;
  const cudaError_t e = D == 128 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bwd_delta_kernel<128>, 256, 0)
                                 : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bwd_delta_kernel<64>, 256, 0);
  return (e != cudaSuccess || per_sm < 1) ? 1 : per_sm;
}
namespace {

size_t rows_bytes(const l2a_params* p) { return align_up((size_t)p->B * p->Lq * p->Hq * p->D * sizeof(bf16), 256); }
size_t stat_bytes(const l2a_params* p) { return align_up((size_t)p->B * p->Hq * p->Lq * sizeof(float), 256); }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace

int bwd_ranges(int n_kblocks, int n_events, int first[kMaxBwdRanges]) {
  first[0] = 0;
  if (n_events >= 11 && n_kblocks >= 16) {
    first[1] = n_kblocks / 2; first[2] = (3 * n_kblocks) / 4; first[3] = (7 * n_kblocks) / 8;
    return 4;
  }
  if (n_events >= 7 && n_kblocks >= 8) {
    first[1] = (3 * n_kblocks) / 4;
    return 2;
  }
  return 1;
}

// First row tile whose dQ still receives contributions from the key blocks at or after `split`: a row at position p
// only meets keys <= p, so after the key blocks below `split` the rows with p < 128 * split are final.
int dq_final_tiles(int split, int q_pos_offset, int n_tiles) {
  const long long rows = (long long)split * kTileN - q_pos_offset;
  if (rows <= 0) return 0;
  const long long t = rows / kTileM;
  return t > n_tiles ? n_tiles : (int)t;
}

template <int D>
cudaError_t launch_bwd(const BwdArgs& base, const CUtensorMap& mapQ, const CUtensorMap& mapDO,
                       const CUtensorMap& mapQc, const CUtensorMap& mapDOc, const CUtensorMap& mapK,
                       const CUtensorMap& mapV, const uint8_t* d_mask, cudaStream_t s) {
  const DeviceInfo* dev = device_info();
  if (dev == nullptr) return cudaErrorUnknown;
  static PerDeviceOnce once;
  cudaError_t e = once.run([] {
    return cudaFuncSetAttribute(bwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<D>::kTotal);
  });
  if (e != cudaSuccess) return e;
  const int n_tiles = (base.Lq + kTileM - 1) / kTileM;
  dq_zero_kernel<<<dev->sms * 8, 256, 0, s>>>(base.dq_acc_loc, base.dq_acc_glb, base.n_routed, base.B, base.Hq, n_tiles,
                                              kTileM * D);
  phase_events().mark(s);
  const int n_kblocks = (base.Lk + kTileN - 1) / kTileN;
  // A caller that registered phase events for key-block ranges wants the gradients of the early rows while the rest is
  // computed (to move them to the host): one launch per range, each followed by the merge of the dQ rows it finishes.
  int first[kMaxBwdRanges];
  const int n_ranges = bwd_ranges(n_kblocks, phase_events().n, first);
  int t_done = 0;
  for (int part = 0; part < n_ranges; ++part) {
    BwdArgs a = base;
    const int kb_end = part + 1 < n_ranges ? first[part + 1] : n_kblocks;
    a.kb_begin = first[part];
    a.kb_count = kb_end - first[part];
    bwd_kernel<D><<<(unsigned)a.kb_count * base.B * base.Hkv, kDkvThreads, BwdSmem<D>::kTotal, s>>>(
        mapQ, mapDO, mapQc, mapDOc, mapK, mapV, a);
    phase_events().mark(s);
    const int t1 = part + 1 < n_ranges ? dq_final_tiles(kb_end, base.q_pos_offset, n_tiles) : n_tiles;
    if (t1 > t_done)
      dq_merge_kernel<D><<<(unsigned)((t1 - t_done) * base.B * base.Hq), 256, 0, s>>>(
          base.dq_acc_loc, base.dq_acc_glb, d_mask, base.prefix, base.dQ, base.B, base.Lq, base.Hq, base.scale,
          base.dq_st.b, base.dq_st.t, t_done, t1 - t_done, base.status);
    if (t1 > t_done) t_done = t1;
    phase_events().mark(s);
  }
  return cudaGetLastError();
}

// one fp32 dQ accumulator: whole 128-row tiles
size_t acc_bytes(const l2a_params* p) {
  return align_up((size_t)p->B * p->Hq * ceil_div(p->Lq, kTileM) * kTileM * p->D * sizeof(float), 256);
}
size_t bwd_ws_size(const l2a_params* p) { return kWsHeaderBytes + 2 * rows_bytes(p) + 3 * stat_bytes(p) + 2 * acc_bytes(p); }

}  // namespace l2a

using namespace l2a;

extern "C" l2a_status l2a_backward(const l2a_params* p, const void* Q, const void* K, const void* V,
                                   const uint8_t* d_mask, const int32_t* q_idx, const int32_t* n_routed,
                                   const int32_t* prefix, const void* dO, const void* S_save, const void* A_c,
                                   const float* lse_loc, const float* lse_glb, void* dQ, void* dK, void* dV,
                                   float* dgate, void* bwd_ws, size_t bwd_ws_bytes, void* stream) {
  return l2a_backward_split(p, Q, K, V, d_mask, q_idx, n_routed, prefix, dO, dO, S_save, A_c, lse_loc, lse_glb, dQ, dK,
                            dV, dgate, bwd_ws, bwd_ws_bytes, stream);
}

static l2a_status backward_impl(const l2a_params* p, const void* Q, const void* K, const void* V,
                                const uint8_t* d_mask, const int32_t* q_idx, const int32_t* n_routed,
                                const int32_t* prefix, const void* dO, const void* dS_loc, const void* S_save,
                                const void* A_c, const float* lse_loc, const float* lse_glb, void* dQ, void* dK,
                                void* dV, float* dgate, void* bwd_ws, size_t bwd_ws_bytes, void* stream,
                                bool clear_status);

extern "C" l2a_status l2a_backward_split(const l2a_params* p, const void* Q, const void* K, const void* V,
                                         const uint8_t* d_mask, const int32_t* q_idx, const int32_t* n_routed,
                                         const int32_t* prefix, const void* dO, const void* dS_loc,
                                         const void* S_save, const void* A_c, const float* lse_loc,
                                         const float* lse_glb, void* dQ, void* dK, void* dV, float* dgate,
                                         void* bwd_ws, size_t bwd_ws_bytes, void* stream) {
  return backward_impl(p, Q, K, V, d_mask, q_idx, n_routed, prefix, dO, dS_loc, S_save, A_c, lse_loc, lse_glb, dQ, dK,
                       dV, dgate, bwd_ws, bwd_ws_bytes, stream, true);
}

// Section 3.1: in the paper's layer Global Attention has its own projections of the local output, i.e. its own
// Q/K/V.  One call for both modules: the local module's backward on (Q, K, V), the global module's on (Qg, Kg, Vg).
extern "C" l2a_status l2a_backward_sets(const l2a_params* p, const void* Q, const void* K, const void* V, const void* Qg,
                                        const void* Kg, const void* Vg, const uint8_t* d_mask, const int32_t* q_idx,
                                        const int32_t* n_routed, const int32_t* prefix, const void* dO,
                                        const void* S_save, const void* A_c, const float* lse_loc, const float* lse_glb,
                                        void* dQ, void* dK, void* dV, void* dQg, void* dKg, void* dVg, float* dgate,
                                        void* bwd_ws, size_t bwd_ws_bytes, void* stream) {
  if (!p) return L2A_ERR_INVALID_ARG;
  if (!Qg && !Kg && !Vg)     // one set feeds both modules
    return l2a_backward(p, Q, K, V, d_mask, q_idx, n_routed, prefix, dO, S_save, A_c, lse_loc, lse_glb, dQ, dK, dV, dgate,
                        bwd_ws, bwd_ws_bytes, stream);
  if (!Qg || !Kg || !Vg || !dQg || !dKg || !dVg) return L2A_ERR_INVALID_ARG;
  if (p->flags & (L2A_FLAG_SKIP_LOCAL | L2A_FLAG_SKIP_GLOBAL | L2A_FLAG_FORCE_ALL_GLOBAL)) return L2A_ERR_INVALID_ARG;
  l2a_params q = *p;
  q.flags = (p->flags & ~L2A_FLAG_SHARED_WINDOW) | L2A_FLAG_SKIP_GLOBAL;
  l2a_status st = backward_impl(&q, Q, K, V, nullptr, nullptr, nullptr, nullptr, dO, dO, S_save, nullptr, lse_loc, nullptr,
                                dQ, dK, dV, nullptr, bwd_ws, bwd_ws_bytes, stream, true);
  if (st != L2A_OK) return st;
  q.flags = (p->flags & ~L2A_FLAG_SHARED_WINDOW) | L2A_FLAG_SKIP_LOCAL;
  return backward_impl(&q, Qg, Kg, Vg, d_mask, q_idx, n_routed, prefix, dO, dO, nullptr, A_c, nullptr, lse_glb, dQg, dKg,
                       dVg, dgate, bwd_ws, bwd_ws_bytes, stream, false);
}

static l2a_status backward_impl(const l2a_params* p, const void* Q, const void* K, const void* V,
                                const uint8_t* d_mask, const int32_t* q_idx, const int32_t* n_routed,
                                const int32_t* prefix, const void* dO, const void* dS_loc, const void* S_save,
                                const void* A_c, const float* lse_loc, const float* lse_glb, void* dQ, void* dK,
                                void* dV, float* dgate, void* bwd_ws, size_t bwd_ws_bytes, void* stream,
                                bool clear_status) {
  if (!p) return L2A_ERR_INVALID_ARG;
  if (!dS_loc || !aligned16(dS_loc)) return L2A_ERR_INVALID_ARG;
  size_t need = 0;
  l2a_status st = l2a_workspace_bytes(p, nullptr, nullptr, &need);
  if (st != L2A_OK) return st;
  const bool skip_local = p->flags & L2A_FLAG_SKIP_LOCAL, skip_global = p->flags & L2A_FLAG_SKIP_GLOBAL;
  if (skip_local && skip_global) return L2A_ERR_INVALID_ARG;
  const bool force_all = p->flags & L2A_FLAG_FORCE_ALL_GLOBAL;
  if (!Q || !K || !V || !dO || !dQ || !dK || !dV) return L2A_ERR_INVALID_ARG;
  if (!skip_global && (!d_mask || !q_idx || !n_routed || !prefix || !A_c || !lse_glb)) return L2A_ERR_INVALID_ARG;
  if (!skip_local && (!S_save || !lse_loc)) return L2A_ERR_INVALID_ARG;
  if (force_all && (skip_local || skip_global)) return L2A_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(dO) || !aligned16(S_save) || !aligned16(A_c) ||
      !aligned16(dQ) || !aligned16(dK) || !aligned16(dV))
    return L2A_ERR_INVALID_ARG;
  if (!bwd_ws || (reinterpret_cast<uintptr_t>(bwd_ws) % 256) != 0 || bwd_ws_bytes < need) return L2A_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(bwd_ws);
  if (clear_status && cudaMemsetAsync(ws, 0, kWsHeaderBytes, s) != cudaSuccess) return L2A_ERR_CUDA;
  bf16* Qc = reinterpret_cast<bf16*>(ws + kWsHeaderBytes);
  bf16* dOc = reinterpret_cast<bf16*>(ws + kWsHeaderBytes + rows_bytes(p));
  float* delta_loc = reinterpret_cast<float*>(ws + kWsHeaderBytes + 2 * rows_bytes(p));
  float* delta_glb = reinterpret_cast<float*>(ws + kWsHeaderBytes + 2 * rows_bytes(p) + stat_bytes(p));
  float* lse_c = reinterpret_cast<float*>(ws + kWsHeaderBytes + 2 * rows_bytes(p) + 2 * stat_bytes(p));
  float* dq_acc_loc = reinterpret_cast<float*>(ws + kWsHeaderBytes + 2 * rows_bytes(p) + 3 * stat_bytes(p));
  float* dq_acc_glb = reinterpret_cast<float*>(ws + kWsHeaderBytes + 2 * rows_bytes(p) + 3 * stat_bytes(p) + acc_bytes(p));
  // Shared-window backward: the window's share of a routed row's global gradient rides on the local items (see
  // bwd_delta_kernel).  Needs the same gradient for both outputs; the flag permits it, other modes just ignore it.
  const bool share = (p->flags & L2A_FLAG_SHARED_WINDOW) && dS_loc == dO && !skip_local && !skip_global &&
                     !force_all;

  CUtensorMap mapQ, mapDO, mapQc, mapDOc, mapK, mapV;
  const RowStrides qs = resolve_strides(p->q_stride, p->Lq, p->Hq * p->D);
  const RowStrides ks = resolve_strides(p->k_stride, p->Lk, p->Hkv * p->D);
  const RowStrides vs = resolve_strides(p->v_stride, p->Lk, p->Hkv * p->D);
  const RowStrides os = resolve_strides(p->o_stride, p->Lq, p->Hq * p->D);
  if (!encode_rows_map(&mapQ, Q, p->B, p->Lq, p->Hq * p->D, kTileM, p->D, qs.b, qs.t) ||
      !encode_rows_map(&mapDO, dS_loc, p->B, p->Lq, p->Hq * p->D, kTileM, p->D, os.b, os.t) ||   // local items: dL/ds_t
      !encode_rows_map(&mapQc, Qc, p->B, p->Lq, p->Hq * p->D, kTileM, p->D) ||
      !encode_rows_map(&mapDOc, dOc, p->B, p->Lq, p->Hq * p->D, kTileM, p->D) ||
      !encode_rows_map(&mapK, K, p->B, p->Lk, p->Hkv * p->D, kTileN, p->D, ks.b, ks.t) ||
      !encode_rows_map(&mapV, V, p->B, p->Lk, p->Hkv * p->D, kTileN, p->D, vs.b, vs.t))
    return L2A_ERR_CUDA;

  PhaseEvents& pe = phase_events();
  struct ClearOnExit { PhaseEvents& p; ~ClearOnExit() { p.clear(); } } clear_on_exit{pe};
  pe.mark(s);
  if (!skip_global) {
    if (launch_gather_rows(static_cast<const bf16*>(Q), Qc, q_idx, n_routed, p->B, p->Lq, p->Hq * p->D, s, nullptr, 0,
                           0, qs, reinterpret_cast<int*>(ws)) != cudaSuccess)
      return L2A_ERR_CUDA;
    if (launch_gather_rows(static_cast<const bf16*>(dO), dOc, q_idx, n_routed, p->B, p->Lq, p->Hq * p->D, s, nullptr,
                           0, 0, os, reinterpret_cast<int*>(ws)) != cudaSuccess)
      return L2A_ERR_CUDA;
  }
  pe.mark(s);
  {
    // one resident wave of 8-warp CTAs; the warps take the tokens round-robin
    const DeviceInfo* dev = device_info();
    if (dev == nullptr) return L2A_ERR_CUDA;
    auto kern = p->D == 128 ? bwd_delta_kernel<128> : bwd_delta_kernel<64>;
    int64_t blocks = (int64_t)dev->sms * (p->D == 128 ? dev->delta_ctas_128 : dev->delta_ctas_64);
    const int64_t max_blocks = ((int64_t)p->B * p->Lq + 7) / 8;
    if (blocks > max_blocks) blocks = max_blocks;
    kern<<<(unsigned)blocks, 256, 0, s>>>(static_cast<const bf16*>(dO), static_cast<const bf16*>(dS_loc),
                                          static_cast<const bf16*>(skip_local ? nullptr : S_save),
                                          static_cast<const bf16*>(A_c), skip_global ? nullptr : d_mask, prefix,
                                          delta_loc, delta_glb, dgate, p->B, p->Lq, p->Hq,
                                          force_all ? 1 : 0, os.b, os.t, lse_loc, lse_glb, share ? lse_c : nullptr);
    if (cudaGetLastError() != cudaSuccess) return L2A_ERR_CUDA;
    if (force_all) {
      dim3 grid((p->Lq + 255) / 256, p->Hq, p->B);
      compact_stat_kernel<<<grid, 256, 0, s>>>(lse_glb, lse_c, q_idx, n_routed, p->Lq, p->Hq);
      if (cudaGetLastError() != cudaSuccess) return L2A_ERR_CUDA;
    }
  }
  BwdArgs a;
  a.B = p->B; a.Lq = p->Lq; a.Lk = p->Lk; a.Hq = p->Hq; a.Hkv = p->Hkv; a.D = p->D;
  a.window = p->window < (1 << 30) ? p->window : (1 << 30);   // any window >= Lk is the same
  a.q_pos_offset = p->q_pos_offset;
  a.scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->D);
  a.scale_log2 = a.scale * kLog2e;
  a.skip_local = skip_local ? 1 : 0;
  a.skip_global = skip_global ? 1 : 0;
  a.q_idx = q_idx; a.n_routed = n_routed; a.prefix = prefix;
  a.seq_bounds = p->seq_bounds;
  a.lse_loc = share ? lse_c : lse_loc; a.lse_glb = force_all ? lse_c : lse_glb;
  a.vis_shift = share ? (p->window < (1 << 30) ? p->window : (1 << 30)) + 1 : 0; a.delta_loc = delta_loc; a.delta_glb = delta_glb;
  a.dQ = static_cast<bf16*>(dQ); a.dK = static_cast<bf16*>(dK); a.dV = static_cast<bf16*>(dV);
  a.dq_st = qs; a.dk_st = ks; a.dv_st = vs;
  a.dq_acc_loc = !skip_local ? dq_acc_loc : nullptr;
  a.dq_acc_glb = !skip_global ? dq_acc_glb : nullptr;
  a.status = reinterpret_cast<int*>(ws);
  const cudaError_t e =
      p->D == 128 ? launch_bwd<128>(a, mapQ, mapDO, mapQc, mapDOc, mapK, mapV, skip_global ? nullptr : d_mask, s)
                  : launch_bwd<64>(a, mapQ, mapDO, mapQc, mapDOc, mapK, mapV, skip_global ? nullptr : d_mask, s);
  return e == cudaSuccess ? L2A_OK : L2A_ERR_CUDA;
}
