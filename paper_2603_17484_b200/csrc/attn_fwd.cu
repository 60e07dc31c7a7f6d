// Forward attention kernel for sm_100a: one kernel, two modes.
//
//   local  mode (Eq. 2, sliding-window mask of Section 2): query rows are sequence rows; key blocks
//          wholly outside the band [p - W, p] are never loaded.
//   global mode (Eq. 4; Algorithm 1): query rows are the compacted routed rows (Q_c); the causal
//          mask uses the true position Q_idx of each compact row; the key loop of a tile stops at
//          the block holding its largest position; the epilogue scatters the result to O by
//          position and combines it with the local output already there (Eq. 5), and also stores
//          the compact output O_c and log-sum-exp L_c.
//
// Structure (per CTA: two 128-row query tiles of one head, sharing the K/V stream):
//   warps 0-7       : soft-max + correction + epilogue.  Warpgroup t (4 warps) owns tile t; one thread per query
//                     row (= TMEM lane) holds the row's 128 scores of a key block in registers, so the row maximum
//                     and the row sum need no exchange between threads.
//   warp 8          : TMA producer (Q once; K and V blocks through 2-stage rings)
//   warp 9          : tcgen05 MMA issuer and TMEM owner
//   TMEM (512 cols) : S0 | S1 | O0 | O1 (fp32); the bf16 probabilities P overwrite the first half
//                     of their own S columns and are consumed from TMEM as the A operand of P*V.
// While one tile's soft-max runs on the CUDA cores, the tensor core works on the other tile.
// The online soft-max follows Algorithm 1 (running max m, running sum l, rescaled accumulator),
// in the exp2 domain, with the rescale skipped while the maximum grows by less than 2^8.
#include "l2a_common.cuh"
#include "sm100_prims.cuh"

namespace l2a {

namespace {

constexpr int kNumTiles = 2;
constexpr int kStages = 2;
constexpr int kSoftmaxWarps = 8;
constexpr int kTmaWarp = kSoftmaxWarps, kMmaWarp = kSoftmaxWarps + 1;
// Twelve warps start with 168 registers each (warps are allocated four at a time, so ten would cost the same); the
// warpgroup of the TMA, MMA and two idle warps hands most of its share to the soft-max warps.
constexpr int kFwdThreads = (kSoftmaxWarps + 4) * 32;   // 384
constexpr int kSoftmaxRegs = 216, kOtherRegs = 72;
static_assert(kSoftmaxWarps * kSoftmaxRegs + 4 * kOtherRegs <= (kSoftmaxWarps + 4) * 168, "register shares exceed the launch allocation");
constexpr float kRescaleThreshold = 8.0f;  // log2 units

template <int D>
struct FwdSmem {
  static constexpr int kQTileBytes = kTileM * D * 2;
  static constexpr int kKVTileBytes = kTileN * D * 2;
  static constexpr int kBoxBytes = 128 * 128;  // one TMA box: 128 rows x 64 bf16 (128 B)
  static constexpr int kQOff = 0;
  static constexpr int kKOff = kQOff + kNumTiles * kQTileBytes;
  static constexpr int kVOff = kKOff + kStages * kKVTileBytes;
  static constexpr int kBarOff = kVOff + kStages * kKVTileBytes;
  static constexpr int kTotal = kBarOff + 256 + 1024 /* alignment slack */;
};

struct Barriers {
  uint64_t q_full[kNumTiles];
  uint64_t k_full[kStages], k_empty[kStages];
  uint64_t v_full[kStages], v_empty[kStages];
  uint64_t s_full[kNumTiles];
  uint64_t p_full[kNumTiles];
  uint64_t o_final;
  uint32_t tmem_base;
  int abort_flag;
};

struct TileRange {
  int active;    // tile has at least one valid row
  int min_pos, max_pos;
  int max_lo;    // largest "first visible key position" among the rows (the last row's)
  int lo, hi;    // first / last key block
};

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                const __grid_constant__ CUtensorMap mapV, const FwdArgs a) {
  using SM = FwdSmem<D>;
  constexpr int kKSteps = D / 16;      // MMA k-steps of Q*K^T
  constexpr int kOCol0 = 2 * kTileN;   // first TMEM column of the O accumulators

  // ---- work item: heaviest first (largest row index first), heads fastest for K/V reuse in L2
  const int h = blockIdx.x % a.Hq;
  const int rest = blockIdx.x / a.Hq;
  const int b = rest % a.B;
  const int pi = a.pair_end - 1 - rest / a.B;
  const int g = h / (a.Hq / a.Hkv);
  const bool compact = a.global_mode && !a.all_rows;           // rows are compact indices into q_idx
  const int n_rows = compact ? a.n_routed[b] : a.Lq;           // valid (compact) rows of this batch entry
  const int row0 = pi * kRowsPerCta;
  if (row0 >= n_rows) return;

  const int32_t* q_idx_b = a.q_idx + (int64_t)b * a.Lq;
  const int w_eff = a.global_mode ? 0x3fffffff : a.window;
  // shared-window mode: a row at position p attends to the keys 0 .. p - W - 1 only (the window p - W .. p is the
  // local pass's share and enters in the epilogue)
  const bool shared = a.global_mode && a.shared_window;
  const int vis_shift = shared ? a.window + 1 : 0;
  if (a.global_mode) {
    // launches restricted to a row range take the groups whose last row falls into it: every group exactly once
    const int c_last = min(row0 + kRowsPerCta, n_rows) - 1;
    const int t_last = compact ? q_idx_b[c_last] : c_last;
    if (t_last < a.row_begin || t_last >= a.row_end) return;
  }

  TileRange tr[kNumTiles];
  int jlo = 0x7fffffff, jhi = -1;
#pragma unroll
  for (int t = 0; t < kNumTiles; ++t) {
    const int first = row0 + t * kTileM;
    int last = first + kTileM - 1;
    if (last > n_rows - 1) last = n_rows - 1;
    tr[t].active = first < n_rows;
    if (tr[t].active) {
      const int first_seq = compact ? q_idx_b[first] : first, last_seq = compact ? q_idx_b[last] : last;
      tr[t].min_pos = first_seq + a.q_pos_offset;
      tr[t].max_pos = last_seq + a.q_pos_offset;
      int lo_pos = tr[t].min_pos - w_eff;
      tr[t].max_lo = tr[t].max_pos - w_eff;
      if (a.seq_bounds != nullptr) {
        // packed sequences: no key before the start of the row's own sequence (starts ascend with the rows)
        lo_pos = max(lo_pos, a.seq_bounds[2 * first_seq]);
        tr[t].max_lo = max(tr[t].max_lo, a.seq_bounds[2 * last_seq]);
      }
      const int hi_pos = tr[t].max_pos - vis_shift;   // last key position any row of the tile attends to
      if (hi_pos >= 0 && hi_pos >= lo_pos) {
        tr[t].lo = lo_pos > 0 ? lo_pos / kTileN : 0;
        tr[t].hi = hi_pos / kTileN;
        jlo = min(jlo, tr[t].lo);
        jhi = max(jhi, tr[t].hi);
      } else {
        tr[t].lo = 1; tr[t].hi = 0;   // shared-window mode: every key of these rows lies inside the window
      }
    } else {
      tr[t].min_pos = tr[t].max_pos = tr[t].max_lo = 0;
      tr[t].lo = 1; tr[t].hi = 0;
    }
  }

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem + SM::kQOff;
  uint8_t* sK = smem + SM::kKOff;
  uint8_t* sV = smem + SM::kVOff;
  Barriers* bar = reinterpret_cast<Barriers*>(smem + SM::kBarOff);
  volatile int* abort_flag = &bar->abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int t = 0; t < kNumTiles; ++t) {
      mbar_init(&bar->q_full[t], 1);
      mbar_init(&bar->s_full[t], 1);
      mbar_init(&bar->p_full[t], kTileM);
    }
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bar->k_full[s], 1);
      mbar_init(&bar->k_empty[s], 1);
      mbar_init(&bar->v_full[s], 1);
      mbar_init(&bar->v_empty[s], 1);
    }
    mbar_init(&bar->o_final, 1);
    bar->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == kMmaWarp) {
    tmem_alloc(&bar->tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bar->tmem_base;
  if (tmem != 0) {
    // all 512 columns were requested, so the allocation must start at column 0; the MMA warp relies on it to
    // keep its TMEM operand addresses compile-time constants
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tmem, 512);
    if (tid == 0) atomicExch(a.status, 3);
    return;
  }

  if (warp == kTmaWarp) {
    // =========================================================================== TMA producer
    setmaxnreg_dec<kOtherRegs>();
    if (lane == 0) {
      tma_prefetch_desc(&mapQ);
      tma_prefetch_desc(&mapK);
      tma_prefetch_desc(&mapV);
      for (int t = 0; t < kNumTiles; ++t) {
        if (!tr[t].active || tr[t].lo > tr[t].hi) continue;
        mbar_expect_tx(&bar->q_full[t], SM::kQTileBytes);
        tma_load_4d(sQ + t * SM::kQTileBytes, &mapQ, &bar->q_full[t], 0, row0 + t * kTileM, h * (D / 64), b);
      }
      for (int j = jlo; j <= jhi; ++j) {
        const int it = j - jlo, s = it % kStages;
        const uint32_t ph = (it / kStages) & 1;
        if (!mbar_wait(&bar->k_empty[s], ph ^ 1, abort_flag)) break;
        mbar_expect_tx(&bar->k_full[s], SM::kKVTileBytes);
        tma_load_4d(sK + s * SM::kKVTileBytes, &mapK, &bar->k_full[s], 0, j * kTileN, g * (D / 64), b);
        if (!mbar_wait(&bar->v_empty[s], ph ^ 1, abort_flag)) break;
        mbar_expect_tx(&bar->v_full[s], SM::kKVTileBytes);
        tma_load_4d(sV + s * SM::kKVTileBytes, &mapV, &bar->v_full[s], 0, j * kTileN, g * (D / 64), b);
      }
    }
    __syncwarp();
  } else if (warp == kMmaWarp) {
    // =========================================================================== MMA issuer
    setmaxnreg_dec<kOtherRegs>();
    // The whole warp runs this loop (uniform control flow keeps the descriptor arithmetic in uniform registers);
    // only the tcgen05 instructions themselves are predicated on lane 0.  Operand descriptors are built once per
    // tile / stage and advanced by compile-time constants, so that issuing stays well under the 64 clocks one
    // 128x128x16 MMA takes.
    {
      const uint32_t leader = (lane == 0);
      constexpr uint32_t tmem = 0;   // checked above: TMEM operand addresses are immediates in this loop
      static_assert(kStages == 2 && kNumTiles == 2, "descriptor selects below assume two stages and two tiles");
      constexpr uint32_t idesc_qk = idesc_bf16_f32(kTileM, kTileN, 0, 0);
      constexpr uint32_t idesc_pv = idesc_bf16_f32(kTileM, D, 0, 1);
      const uint64_t dq0 = smem_desc_sw128(smem_u32(sQ), 16, 1024);
      const uint64_t dq1 = smem_desc_sw128(smem_u32(sQ + SM::kQTileBytes), 16, 1024);
      const uint64_t dk0 = smem_desc_sw128(smem_u32(sK), 16, 1024);
      const uint64_t dk1 = smem_desc_sw128(smem_u32(sK + SM::kKVTileBytes), 16, 1024);
      const uint64_t dv0 = smem_desc_sw128(smem_u32(sV), SM::kBoxBytes, 1024);
      const uint64_t dv1 = smem_desc_sw128(smem_u32(sV + SM::kKVTileBytes), SM::kBoxBytes, 1024);
      const int lo0 = tr[0].lo, hi0 = tr[0].hi, lo1 = tr[1].lo, hi1 = tr[1].hi;  // an inactive tile has lo > hi
      uint32_t p_cnt0 = 0, p_cnt1 = 0;
      bool ok = true;

      auto issue_qk = [&](int t, int s) {
        const uint64_t qd = t ? dq1 : dq0, kd = s ? dk1 : dk0;
        const uint32_t d = tmem + t * kTileN;
#pragma unroll
        for (int kk = 0; kk < kKSteps; ++kk) {
          const uint32_t c = ((kk >> 2) * SM::kBoxBytes + (kk & 3) * 32) >> 4;
          mma_ss(d, qd + c, kd + c, idesc_qk, kk > 0, leader);
        }
        tc_commit(&bar->s_full[t], leader);
      };
      auto issue_pv = [&](int t, int s, uint32_t acc) {
        const uint64_t vd = s ? dv1 : dv0;
        const uint32_t d = tmem + kOCol0 + t * D, p = tmem + t * kTileN;
#pragma unroll
        for (int kk = 0; kk < kTileN / 16; ++kk)
          mma_ts(d, p + (kk >> 2) * 64 + (kk & 3) * 8, vd + ((kk * 2048) >> 4), idesc_pv, kk > 0 ? 1u : acc, leader);
      };
      auto in_range = [&](int t, int j) { return t ? (j >= lo1 && j <= hi1) : (j >= lo0 && j <= hi0); };

      if (jhi < jlo) ok = false;   // no key block at all (shared-window mode): nothing to issue, nobody waits
      // first key block: Q*K^T for both tiles
      if (ok && !mbar_spin_warp(&bar->k_full[0], 0, abort_flag)) ok = false;
#pragma unroll
      for (int t = 0; t < kNumTiles; ++t) {
        if (ok && in_range(t, jlo)) {
          if (!mbar_spin_warp(&bar->q_full[t], 0, abort_flag)) { ok = false; }
          else { tc_fence_after(); issue_qk(t, 0); }
        }
      }
      if (ok) tc_commit(&bar->k_empty[0], leader);

      for (int j = jlo; ok && j <= jhi; ++j) {
        const int it = j - jlo, s = it & 1, sn = s ^ 1;
        const uint32_t ph = (it >> 1) & 1;
        const uint32_t phn = ((it + 1) >> 1) & 1;
        bool v_ready = false, k_ready = false;
#pragma unroll
        for (int t = 0; t < kNumTiles; ++t) {
          if (ok && in_range(t, j)) {
            uint32_t& pc = t ? p_cnt1 : p_cnt0;
            if (!mbar_spin_warp(&bar->p_full[t], pc & 1, abort_flag)) { ok = false; }
            else {
              ++pc;
              if (!v_ready) {
                if (!mbar_spin_warp(&bar->v_full[s], ph, abort_flag)) ok = false;
                v_ready = true;
              }
              if (ok) {
                tc_fence_after();
                issue_pv(t, s, j > (t ? lo1 : lo0) ? 1u : 0u);
              }
            }
          }
          if (ok && j + 1 <= jhi && in_range(t, j + 1)) {
            if (!k_ready) {
              if (!mbar_spin_warp(&bar->k_full[sn], phn, abort_flag)) ok = false;
              k_ready = true;
            }
            if (ok && j + 1 == (t ? lo1 : lo0) && !mbar_spin_warp(&bar->q_full[t], 0, abort_flag)) ok = false;
            if (ok) {
              tc_fence_after();
              issue_qk(t, sn);
            }
          }
        }
        if (!ok) break;
        // V block j is released once both tiles' P*V have drained; K block j+1 once both Q*K^T have
        if (!v_ready && !mbar_spin_warp(&bar->v_full[s], ph, abort_flag)) break;
        tc_commit(&bar->v_empty[s], leader);
        if (j + 1 <= jhi) {
          if (!k_ready && !mbar_spin_warp(&bar->k_full[sn], phn, abort_flag)) break;
          tc_commit(&bar->k_empty[sn], leader);
        }
      }
      if (ok) tc_commit(&bar->o_final, leader);
    }
    __syncwarp();
  } else if (warp > kMmaWarp) {
    setmaxnreg_dec<kOtherRegs>();     // idle warps of the fourth warpgroup
  } else {
    // =========================================================================== soft-max warpgroups
    setmaxnreg_inc<kSoftmaxRegs>();
    const int t = warp >> 2;                 // tile of this warpgroup
    const int r = (warp & 3) * 32 + lane;    // row inside the tile == TMEM lane
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t s_addr = tmem + lane_base + t * kTileN;        // this row's 128 score columns
    const uint32_t o_addr = tmem + lane_base + kOCol0 + t * D;    // its D accumulator columns
    const TileRange my = t ? tr[1] : tr[0];
    if (my.active) {
      const int row = row0 + t * kTileM + r;           // sequence row (local) or compact row (global)
      const bool valid = row < n_rows;
      const int seq_row = valid ? (compact ? q_idx_b[row] : row) : -1;
      const int pos = valid ? seq_row + a.q_pos_offset - vis_shift : -1;   // largest visible key position
      int pos_lo = valid ? (pos - w_eff) : 0x7fffffff;                     // smallest visible key position
      if (valid && a.seq_bounds != nullptr) pos_lo = max(pos_lo, a.seq_bounds[2 * seq_row]);
      float m_use = -INFINITY;   // reference maximum, exp2 domain
      float l = 0.f;             // row sum
      bool ok = true;
      const int n_my = my.hi - my.lo + 1;

      for (int i = 0; i < n_my; ++i) {
        const int j = my.lo + i;
        // warp-uniform outcome: the TMEM loads/stores below are warp-collective
        if (!__all_sync(0xffffffffu, mbar_wait(&bar->s_full[t], i & 1, abort_flag))) { ok = false; break; }
        tc_fence_after();
        const int k0 = j * kTileN;
        const bool partial = (k0 + kTileN - 1 > my.min_pos - vis_shift) || (k0 < my.max_lo);
        uint32_t v[4][32];       // the row's scores of this key block
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(s_addr + c * 32, v[c]);
        tmem_ld_wait();
        if (partial) {
          // edge block (causal diagonal, left window edge, ragged rows): masked scores become -inf, whose
          // exponential is an exact zero below
#pragma unroll
          for (int c = 0; c < 4; ++c) {
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              const int kp = k0 + c * 32 + e;
              v[c][e] = (kp <= pos && kp >= pos_lo) ? v[c][e] : 0xff800000u;
            }
          }
        }
        float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          mx0 = fmax3(mx0, __uint_as_float(v[0][e]), __uint_as_float(v[0][e + 1]));
          mx1 = fmax3(mx1, __uint_as_float(v[1][e]), __uint_as_float(v[1][e + 1]));
          mx2 = fmax3(mx2, __uint_as_float(v[2][e]), __uint_as_float(v[2][e + 1]));
          mx3 = fmax3(mx3, __uint_as_float(v[3][e]), __uint_as_float(v[3][e + 1]));
        }
        const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
        const float m_new = fmaxf(m_use, mx * a.scale_log2);

        // correction: rescale the running sum and the TMEM accumulator only when the maximum moved a lot
        const bool need = (i == 0) ? false : (m_new - m_use > kRescaleThreshold);
        if (i == 0) m_use = m_new;
        if (__any_sync(0xffffffffu, need)) {
          const float alpha = need ? fast_exp2(m_use - m_new) : 1.0f;
          l *= alpha;
#pragma unroll 1
          for (int c = 0; c < D / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(o_addr + c * 32, o);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st32(o_addr + c * 32, o);
          }
          if (need) m_use = m_new;
        }
        const float m_eff = (m_use == -INFINITY) ? 0.f : m_use;
        const float neg_m = -m_eff;
        // probabilities; the bf16 P of keys 64h .. 64h+63 overwrites score columns 64h .. 64h+31
        float2 sum2 = make_float2(0.f, 0.f);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t pk[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float2 x = __ffma2_rn(make_float2(__uint_as_float(v[c][2 * e]), __uint_as_float(v[c][2 * e + 1])),
                                        make_float2(a.scale_log2, a.scale_log2), make_float2(neg_m, neg_m));
            const float2 p = make_float2(fast_exp2(x.x), fast_exp2(x.y));
            sum2 = __fadd2_rn(sum2, p);
            pk[e] = pack_bf16(p.x, p.y);
          }
          tmem_st16(s_addr + (c >> 1) * 64 + (c & 1) * 16, pk);
        }
        l += sum2.x + sum2.y;
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive(&bar->p_full[t]);
      }

      // ---- epilogue: O / l, log-sum-exp, store (local) or scatter + combine (global)
      if (ok && (n_my == 0 || __all_sync(0xffffffffu, mbar_wait(&bar->o_final, 0, abort_flag)))) {
        tc_fence_after();
        float inv_l = (l > 0.f) ? 1.0f / l : 0.f;
        float lse2 = m_use + log2f(l);   // log-sum-exp in the exp2 domain
        float c_loc = 0.f;               // shared-window mode: weight of the local result s_t in a_t
        if (shared && valid) {
          // a_t = (e^{lse_out} o_out + e^{lse_loc} s_t) / (e^{lse_out} + e^{lse_loc}): the softmax over the whole
          // prefix, split into the keys before the window (this kernel) and the window (the local pass)
          const float lse_out2 = (l > 0.f) ? lse2 : -INFINITY;
          const float lse_loc2 = a.lse_loc[((int64_t)b * a.Hq + h) * a.Lq + seq_row] * 1.4426950408889634f;
          const float mm = fmaxf(lse_out2, lse_loc2);
          const float w_out = fast_exp2(lse_out2 - mm), w_loc = fast_exp2(lse_loc2 - mm);
          const float inv = 1.0f / (w_out + w_loc);
          inv_l *= w_out * inv;
          c_loc = w_loc * inv;
          lse2 = mm + log2f(w_out + w_loc);
        }
        if (valid && a.lse != nullptr) {
          const float lse = lse2 * 0.6931471805599453f;
          a.lse[((int64_t)b * a.Hq + h) * a.Lq + row] = lse;
        }
        bf16* dst1 = nullptr;   // row-indexed destination (s rows, or compact a rows)
        bf16* dst2 = nullptr;   // position-indexed destination
        if (valid && dbg_in_range(row >= 0 && row < a.Lq && seq_row >= 0 && seq_row < a.Lq, a.status)) {
          if (a.out) dst1 = a.out + b * a.out_st.b + row * a.out_st.t + (int64_t)h * D;
          if (a.out2 && (a.combine_mask == nullptr || a.combine_mask[(int64_t)b * a.Lq + seq_row]))
            dst2 = a.out2 + b * a.out2_st.b + seq_row * a.out2_st.t + (int64_t)h * D;
        }
        const bool accumulate = a.global_mode && a.accumulate_into_out2;
#pragma unroll 1
        for (int c = 0; c < D / 32; ++c) {
          uint32_t o[32];
          if (n_my > 0) {
            tmem_ld32(o_addr + c * 32, o);
            tmem_ld_wait();
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = 0u;    // no key before the window: the accumulator was never written
          }
          float f[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) f[e] = __uint_as_float(o[e]) * inv_l;
          if (shared && dst2) {
            const uint4* s4 = reinterpret_cast<const uint4*>(dst2 + c * 32);   // s_t, written by the local pass
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint4 old = s4[q];
              const uint32_t ow[4] = {old.x, old.y, old.z, old.w};
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                f[8 * q + 2 * k] = fmaf(c_loc, __uint_as_float(ow[k] << 16), f[8 * q + 2 * k]);
                f[8 * q + 2 * k + 1] = fmaf(c_loc, __uint_as_float(ow[k] & 0xffff0000u), f[8 * q + 2 * k + 1]);
              }
            }
          }
          if (dst1) {
            uint4* d4 = reinterpret_cast<uint4*>(dst1 + c * 32);
#pragma unroll
            for (int q = 0; q < 4; ++q)
              d4[q] = make_uint4(pack_bf16(f[8 * q], f[8 * q + 1]), pack_bf16(f[8 * q + 2], f[8 * q + 3]),
                                 pack_bf16(f[8 * q + 4], f[8 * q + 5]), pack_bf16(f[8 * q + 6], f[8 * q + 7]));
          }
          if (dst2) {
            uint4* d4 = reinterpret_cast<uint4*>(dst2 + c * 32);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              if (accumulate) {
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
  }

  // ---- teardown
  tc_fence_before();
  __syncthreads();
  if (bar->abort_flag) {
    // a bounded wait ran out: give copies still in flight time to land before shared memory is released
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    if (tid == 0) atomicExch(a.status, 1);
    __syncthreads();
  }
  if (warp == kMmaWarp) tmem_dealloc(tmem, 512);
}

}  // namespace

cudaError_t launch_attn_fwd(const FwdArgs& a, const CUtensorMap& mapQ, const CUtensorMap& mapK,
                            const CUtensorMap& mapV, cudaStream_t stream) {
  const unsigned grid = (unsigned)(a.pair_end - a.pair_begin) * a.Hq * a.B;
  if (a.pair_end <= a.pair_begin) return cudaSuccess;
  cudaError_t e;
  if (a.D == 128) {
    static PerDeviceOnce once;
    e = once.run([] {
      return cudaFuncSetAttribute(attn_fwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<128>::kTotal);
    });
    if (e != cudaSuccess) return e;
    attn_fwd_kernel<128><<<grid, kFwdThreads, FwdSmem<128>::kTotal, stream>>>(mapQ, mapK, mapV, a);
  } else {
    static PerDeviceOnce once;
    e = once.run([] {
      return cudaFuncSetAttribute(attn_fwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<64>::kTotal);
    });
    if (e != cudaSuccess) return e;
    attn_fwd_kernel<64><<<grid, kFwdThreads, FwdSmem<64>::kTotal, stream>>>(mapQ, mapK, mapV, a);
  }
  return cudaGetLastError();
}

}  // namespace l2a
