// Internal declarations shared by the translation units of libl2a.so (not part of the C ABI).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/l2a.h"

namespace l2a {

typedef __nv_bfloat16 bf16;

constexpr int kTileM = 128;         // query rows per MMA tile
constexpr int kTileN = 128;         // keys per KV block
constexpr int kRowsPerCta = 256;    // two query tiles per CTA in the forward / dQ kernels
constexpr size_t kWsHeaderBytes = 256;  // every workspace starts with a header; word 0 = status

// Debug build (-DL2A_DEBUG): every index derived from q_idx / prefix / tile metadata is checked against the tensor
// extent before it is used for a store; a violation sets the workspace status word to 4 (l2a_workspace_status then
// returns L2A_ERR_DEVICE_BOUNDS) and the store is skipped -- nothing traps.  In the normal build the check folds away.
#ifdef L2A_DEBUG
__device__ __forceinline__ bool dbg_in_range(bool ok, int* status) {
  if (!ok && status != nullptr) atomicExch(status, 4);
  return ok;
}
#else
__device__ __forceinline__ bool dbg_in_range(bool, int*) { return true; }
#endif

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Host-side: resolved driver entry point for cuTensorMapEncodeTiled, and a helper that encodes a
// [batch, rows, heads*D] bf16 tensor so that ONE copy brings a box_rows x head_dim tile into shared memory in
// the 128-byte-swizzled layout the MMA operand descriptors expect.  Returns false on failure.
bool encode_rows_map(CUtensorMap* map, const void* base, int batch, int rows, int row_elems, int box_rows,
                     int head_dim, int64_t batch_stride = 0, int64_t token_stride = 0);   // strides in elements; 0 = dense

// Strides of a [B, L, H, D] tensor in elements ({batch, token}); heads and head values are contiguous.
struct RowStrides {
  int64_t b, t;
};
inline RowStrides resolve_strides(const int64_t (&s)[2], int L, int row_elems) {
  RowStrides r;
  r.t = s[1] > 0 ? s[1] : row_elems;
  r.b = s[0] > 0 ? s[0] : (int64_t)L * r.t;
  return r;
}
inline bool strides_ok(const int64_t (&s)[2], int L, int row_elems) {
  if (s[0] < 0 || s[1] < 0) return false;
  const RowStrides r = resolve_strides(s, L, row_elems);
  return r.t % 8 == 0 && r.b % 8 == 0 && r.t >= row_elems && r.b >= (int64_t)L * r.t;
}
inline bool is_dense(const int64_t (&s)[2], int L, int row_elems) {
  const RowStrides r = resolve_strides(s, L, row_elems);
  return r.t == row_elems && r.b == (int64_t)L * row_elems;
}

// Launchers (each returns the CUDA error of its launch).  Defined in the kernel files.
struct RouteArgs {
  const void* router;
  int router_kind;
  float threshold;
  int B, L;
  uint8_t* d_mask;
  int32_t* q_idx;
  int32_t* n_routed;
  int32_t* prefix;
  int32_t* block_sums;  // workspace: [B, nblocks]
  int nblocks;
};
constexpr int kRouteBlockElems = 4096;  // positions per CTA of the route/compact kernels
cudaError_t launch_route_compact(const RouteArgs& a, cudaStream_t stream);
cudaError_t launch_pack_sequences(const int32_t* cu_seqlens, int n_seq, int L, int32_t* seq_bounds, cudaStream_t stream);

// Gathers rows src[b, q_idx[b][c], :] -> dst[b, c, :] for c < n_routed[b], and zero-fills rows up to
// the next multiple of kRowsPerCta (bounded by L) so that padded MMA tiles read zeros.  With `prefix` given, only the
// routed rows t in [row_begin, row_end) are gathered (the padding with the range that ends at L).
cudaError_t launch_gather_rows(const bf16* src, bf16* dst, const int32_t* q_idx, const int32_t* n_routed,
                               int B, int L, int row_elems, cudaStream_t stream, const int32_t* prefix = nullptr,
                               int row_begin = 0, int row_end = 0, RowStrides src_strides = RowStrides{0, 0},
                               int* status = nullptr);   // status: workspace status word (debug-build index checks)

// z[b,t] = w . S[b,t,:] + bias (fp32 accumulation); optional sum over t of sigmoid(z)^2 per batch entry
cudaError_t launch_router_logits(const bf16* S, const float* w, float bias, float* logits, float* sum_sq, int B,
                                 int L, int row_elems, cudaStream_t stream);

// Router backward (Eq. 7 with the regulariser's gradient): dz [B,L], dW [row_elems] and dbias [1] (both added with
// atomics to buffers the caller zeroed), dS = dO + dz * w (bf16 rows); dgate, dO/dS, dz, dw, dbias may be NULL.
cudaError_t launch_router_backward(const bf16* S, const float* w, const float* logits, const float* dgate, float coeff,
                                   const bf16* dO, float* dz, float* dw, float* dbias, bf16* dS, int B, int L,
                                   int row_elems, cudaStream_t stream);

struct FwdArgs {
  int B, Lq, Lk, Hq, Hkv, D;
  int window, q_pos_offset;
  float scale_log2;         // softmax_scale * log2(e)
  int global_mode;          // 0: local banded attention over all rows; 1: global attention over compact rows
  int accumulate_into_out2; // global mode: out2[row] = out2[row] + a (1) or out2[row] = a (0)
  int all_rows;             // global mode over EVERY row (identity index list) instead of the compacted ones
  const uint8_t* combine_mask;  // when set, out2 is touched only for rows with a non-zero mask entry
  const int32_t* q_idx;
  const int32_t* n_routed;
  bf16* out;    // local: s rows [B,Lq,Hq,D];  global: compact a rows (A_c) or NULL
  bf16* out2;   // local: optional second copy of s (NULL to skip);  global: O rows, indexed by position
  float* lse;   // local: [B,Hq,Lq] by row;  global: [B,Hq,Lq] by compact row; may be NULL
  int* status;  // workspace status word
  RowStrides out_st, out2_st;   // strides of out / out2 in elements
  int pair_begin, pair_end;  // 256-row query groups [pair_begin, pair_end) this launch covers (all: 0 .. ceil(Lq / 256))
  int row_begin, row_end;    // global mode: only the groups whose LAST row t lies in [row_begin, row_end)
  // Shared-projection fusion (global mode over compact rows): the keys inside the window were already attended by
  // the local pass of the same Q/K/V, so the global pass covers only the keys before the window and merges with the
  // local result (s_t read from out2, its log-sum-exp from lse_loc).
  int shared_window;
  const float* lse_loc;      // [B,Hq,Lq] by row; read only when shared_window is set
  // Packed variable-length batch (B == 1): per token {first token of its sequence, one past the last}; NULL otherwise
  const int32_t* seq_bounds;
};
size_t bwd_ws_size(const l2a_params* p);
// Key-block ranges of the backward when the caller registered phase events for them (11 events: four ranges, 7: two,
// fewer: one launch).  Writes the first key block of ranges 1.. into `first` and returns the number of ranges; ranges
// get shorter towards the end of the sequence, where a key block has little work left.  dq_final_tiles: number of
// leading 128-row tiles of dQ that are final once the key blocks below `split` are done.
constexpr int kMaxBwdRanges = 4;
int bwd_ranges(int n_kblocks, int n_events, int first[kMaxBwdRanges]);
int dq_final_tiles(int split, int q_pos_offset, int n_tiles);

// Facts about the current device that the launchers need, looked up once per device and cached.
struct DeviceInfo {
  int sms;
  int delta_ctas_64, delta_ctas_128;   // resident CTAs per SM of the Delta kernel
};
const DeviceInfo* device_info();       // NULL if the CUDA runtime fails
int delta_ctas_per_sm(int D);          // defined with the backward
// Runs fn() once per device (per call site owning the object): for cudaFuncSetAttribute and the like.
struct PerDeviceOnce {
  static constexpr int kMaxDevices = 64;
  std::atomic<int> done[kMaxDevices];
  PerDeviceOnce() { for (auto& d : done) d.store(0); }
  template <class F>
  cudaError_t run(F fn) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return fn();
    if (done[dev].load(std::memory_order_acquire)) return cudaSuccess;
    e = fn();                         // idempotent: two threads racing here both succeed
    if (e == cudaSuccess) done[dev].store(1, std::memory_order_release);
    return e;
  }
};

// One-shot, thread-local registration of phase-boundary events (see l2a_profile_next_call).
struct PhaseEvents {
  cudaEvent_t ev[12];
  int n = 0;
  int next = 0;
  void mark(cudaStream_t s) {
    if (next < n) cudaEventRecord(ev[next++], s);
  }
  void clear() { n = 0; next = 0; }
};
PhaseEvents& phase_events();  // defined with the backward

cudaError_t launch_attn_fwd(const FwdArgs& a, const CUtensorMap& mapQ, const CUtensorMap& mapK,
                            const CUtensorMap& mapV, cudaStream_t stream);

}  // namespace l2a
