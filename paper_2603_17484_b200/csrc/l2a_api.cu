// C ABI of libl2a.so: argument validation, workspace layout, tensor-map encoding, launch order.
// Every step of the path runs in the CUDA kernels; nothing here computes on the host and there is
// no fallback path.
#include <math.h>
#include <string.h>

#include "l2a_common.cuh"
#include "sm100_prims.cuh"

namespace l2a {

namespace {

typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

encode_tiled_fn get_encode() {
  static encode_tiled_fn fn = []() -> encode_tiled_fn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) return nullptr;
    if (q != cudaDriverEntryPointSuccess) return nullptr;
    return reinterpret_cast<encode_tiled_fn>(p);
  }();
  return fn;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

l2a_status check_params(const l2a_params* p) {
  if (!p) return L2A_ERR_INVALID_ARG;
  if (p->B <= 0 || p->Lq <= 0 || p->Lk <= 0 || p->Hq <= 0 || p->Hkv <= 0 || p->D <= 0) return L2A_ERR_INVALID_ARG;
  if (p->Hq % p->Hkv != 0) return L2A_ERR_INVALID_ARG;
  if (p->window < 0) return L2A_ERR_INVALID_ARG;
  if (p->q_pos_offset < 0 || (int64_t)p->Lq + p->q_pos_offset > p->Lk) return L2A_ERR_INVALID_ARG;
  if (!(p->softmax_scale >= 0.f) || isinf(p->softmax_scale)) return L2A_ERR_INVALID_ARG;
  if ((int64_t)p->B * p->Lq >= (1ll << 31) || (int64_t)p->B * p->Lk >= (1ll << 31)) return L2A_ERR_INVALID_ARG;
  if (p->D != 64 && p->D != 128) return L2A_ERR_UNSUPPORTED;
  if (!strides_ok(p->q_stride, p->Lq, p->Hq * p->D) || !strides_ok(p->k_stride, p->Lk, p->Hkv * p->D) ||
      !strides_ok(p->v_stride, p->Lk, p->Hkv * p->D) || !strides_ok(p->o_stride, p->Lq, p->Hq * p->D))
    return L2A_ERR_INVALID_ARG;
  // packed sequences: one token axis, positions are token indices
  if (p->seq_bounds && (p->B != 1 || p->Lq != p->Lk || p->q_pos_offset != 0 || !aligned(p->seq_bounds, 8)))
    return L2A_ERR_INVALID_ARG;
  return L2A_OK;
}

float scale_of(const l2a_params* p) { return p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->D); }

size_t route_ws_size(const l2a_params* p) {
  const int nblocks = ceil_div(p->Lq, kRouteBlockElems);
  return kWsHeaderBytes + align_up((size_t)p->B * nblocks * sizeof(int32_t), 256);
}
size_t qrows_bytes(const l2a_params* p) { return align_up((size_t)p->B * p->Lq * p->Hq * p->D * sizeof(bf16), 256); }
size_t fwd_ws_size(const l2a_params* p) { return kWsHeaderBytes + qrows_bytes(p); }

bool ws_ok(const void* ws, size_t have, size_t need) { return ws && aligned(ws, 256) && have >= need; }

}  // namespace

PhaseEvents& phase_events() {
  static thread_local PhaseEvents pe;
  return pe;
}

const DeviceInfo* device_info() {
  static DeviceInfo info[PerDeviceOnce::kMaxDevices];
  static PerDeviceOnce once;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= PerDeviceOnce::kMaxDevices) return nullptr;
  const cudaError_t e = once.run([dev] {
    DeviceInfo d;
    cudaError_t r = cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev);
    if (r != cudaSuccess) return r;
    d.delta_ctas_64 = delta_ctas_per_sm(64);
    d.delta_ctas_128 = delta_ctas_per_sm(128);
    info[dev] = d;
    return cudaSuccess;
  });
  return e == cudaSuccess ? &info[dev] : nullptr;
}

bool encode_rows_map(CUtensorMap* map, const void* base, int batch, int rows, int row_elems, int box_rows,
                     int head_dim, int64_t batch_stride, int64_t token_stride) {
  encode_tiled_fn enc = get_encode();
  if (!enc) return false;
  // [batch, rows, row_elems] seen as {64 elements, rows, row_elems / 64 column chunks, batch}: one copy of a
  // {64, box_rows, head_dim / 64, 1} box lands in shared memory as head_dim / 64 consecutive 128-byte-swizzled
  // sub-tiles of box_rows x 64 elements -- the layout the MMA operand descriptors address.
  cuuint64_t dims[4] = {64, (cuuint64_t)rows, (cuuint64_t)(row_elems / 64), (cuuint64_t)batch};
  const int64_t ts = token_stride > 0 ? token_stride : row_elems;
  const int64_t bs = batch_stride > 0 ? batch_stride : (int64_t)rows * ts;
  cuuint64_t strides[3] = {(cuuint64_t)ts * 2, 128, (cuuint64_t)bs * 2};
  cuuint32_t box[4] = {64, (cuuint32_t)box_rows, (cuuint32_t)(head_dim / 64), 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace l2a

using namespace l2a;

extern "C" {

#ifdef L2A_DEBUG
const char* l2a_version(void) { return "l2a-b200 0.2 (sm_100a; tcgen05/TMEM/TMA; debug build: index checks on)"; }
#else
const char* l2a_version(void) { return "l2a-b200 0.2 (sm_100a; tcgen05/TMEM/TMA)"; }
#endif

const char* l2a_status_string(l2a_status s) {
  switch (s) {
    case L2A_OK: return "ok";
    case L2A_ERR_INVALID_ARG: return "invalid argument";
    case L2A_ERR_UNSUPPORTED: return "unsupported configuration";
    case L2A_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case L2A_ERR_CUDA: return "CUDA call failed";
    case L2A_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    case L2A_ERR_DEVICE_BOUNDS: return "an index derived from the routing arrays was out of range (debug build)";
  }
  return "unknown status";
}

l2a_status l2a_workspace_bytes(const l2a_params* p, size_t* route_ws_bytes, size_t* fwd_ws_bytes,
                               size_t* bwd_ws_bytes) {
  l2a_status st = check_params(p);
  if (st != L2A_OK) return st;
  if (route_ws_bytes) *route_ws_bytes = route_ws_size(p);
  if (fwd_ws_bytes) *fwd_ws_bytes = fwd_ws_size(p);
  if (bwd_ws_bytes) *bwd_ws_bytes = l2a::bwd_ws_size(p);
  return L2A_OK;
}

namespace l2a {
namespace {
// The path a kernel takes when one of its waits runs out, on its own: one warp waits (bounded) for an mbarrier
// arrival that never comes, the other warps wait for the first one's outcome through the same abort flag, and the
// CTA records the failure in the status word -- what every kernel of this library does at its end.
__global__ void __launch_bounds__(128) wait_timeout_selftest_kernel(int* status, uint64_t limit_ns) {
  __shared__ uint64_t never_arrives;
  __shared__ uint64_t second;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&never_arrives, 1);
    mbar_init(&second, 1);
    abort_flag = 0;
    fence_mbar_init();
  }
  __syncthreads();
  volatile int* af = &abort_flag;
  const uint64_t second_limit = 1000 * limit_ns < kWaitLimitNs ? 1000 * limit_ns : kWaitLimitNs;
  if (threadIdx.x < 32) mbar_wait(&never_arrives, 0, af, limit_ns);   // gives up after limit_ns, raises the flag
  else mbar_wait(&second, 0, af, second_limit);                        // leaves as soon as the flag is up
  __syncthreads();
  if (threadIdx.x == 0 && abort_flag) atomicExch(status, 1);
}
}  // namespace
}  // namespace l2a

l2a_status l2a_selftest_wait_timeout(void* ws, unsigned limit_us, void* stream) {
  if (!ws || (reinterpret_cast<uintptr_t>(ws) % 256) != 0) return L2A_ERR_WORKSPACE;
  if (limit_us == 0 || limit_us > 1000000u) return L2A_ERR_INVALID_ARG;   // at most one second
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(ws, 0, l2a::kWsHeaderBytes, s) != cudaSuccess) return L2A_ERR_CUDA;
  l2a::wait_timeout_selftest_kernel<<<1, 128, 0, s>>>(static_cast<int*>(ws), (uint64_t)limit_us * 1000ull);
  return cudaGetLastError() == cudaSuccess ? L2A_OK : L2A_ERR_CUDA;
}

l2a_status l2a_workspace_status(const void* ws, void* stream) {
  if (!ws) return L2A_ERR_INVALID_ARG;
  int word = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&word, ws, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return L2A_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return L2A_ERR_CUDA;
  return word == 0 ? L2A_OK : word == 4 ? L2A_ERR_DEVICE_BOUNDS : L2A_ERR_DEVICE_TIMEOUT;
}

l2a_status l2a_pack_sequences(const int32_t* cu_seqlens, int n_seq, int Lq, int32_t* seq_bounds, void* stream) {
  if (!cu_seqlens || !seq_bounds || n_seq < 0 || Lq <= 0 || !aligned(seq_bounds, 8)) return L2A_ERR_INVALID_ARG;
  return launch_pack_sequences(cu_seqlens, n_seq, Lq, seq_bounds, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? L2A_OK : L2A_ERR_CUDA;
}

l2a_status l2a_route_compact(const l2a_params* p, const void* router, int router_kind, float logit_threshold,
                             uint8_t* d_mask, int32_t* q_idx, int32_t* n_routed, int32_t* prefix, void* route_ws,
                             size_t route_ws_bytes, void* stream) {
  l2a_status st = check_params(p);
  if (st != L2A_OK) return st;
  if (!router || !d_mask || !q_idx || !n_routed || !prefix) return L2A_ERR_INVALID_ARG;
  if (router_kind != L2A_ROUTER_MASK_U8 && router_kind != L2A_ROUTER_LOGITS_F32 &&
      router_kind != L2A_ROUTER_LOGITS_BF16)
    return L2A_ERR_INVALID_ARG;
  if (!aligned(q_idx, 4) || !aligned(n_routed, 4) || !aligned(prefix, 4)) return L2A_ERR_INVALID_ARG;
  if (router_kind == L2A_ROUTER_LOGITS_F32 && !aligned(router, 4)) return L2A_ERR_INVALID_ARG;
  if (router_kind == L2A_ROUTER_LOGITS_BF16 && !aligned(router, 2)) return L2A_ERR_INVALID_ARG;
  if (!ws_ok(route_ws, route_ws_bytes, route_ws_size(p))) return L2A_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(route_ws, 0, kWsHeaderBytes, s) != cudaSuccess) return L2A_ERR_CUDA;
  RouteArgs a;
  a.router = router;
  a.router_kind = router_kind;
  a.threshold = logit_threshold;
  a.B = p->B;
  a.L = p->Lq;
  a.d_mask = d_mask;
  a.q_idx = q_idx;
  a.n_routed = n_routed;
  a.prefix = prefix;
  a.block_sums = reinterpret_cast<int32_t*>(static_cast<uint8_t*>(route_ws) + kWsHeaderBytes);
  a.nblocks = ceil_div(p->Lq, kRouteBlockElems);
  return launch_route_compact(a, s) == cudaSuccess ? L2A_OK : L2A_ERR_CUDA;
}

// l2a_forward over the 256-row query groups [pair_begin, pair_end) (pair_end < 0: all of them).  A proper sub-range
// is used by l2a_step_host to start Local Attention on the rows whose queries have already arrived; it is only
// meaningful for the local module (L2A_FLAG_SKIP_GLOBAL), and only the first call of a step clears the status word.
// [row_begin, row_end) restricts the global phase (L2A_FLAG_GLOBAL_PHASE) to the routed rows of that range: the
// gather takes exactly those rows, the attention launch the compact groups whose last row lies in the range.
static l2a_status forward_range(const l2a_params* p, const void* Q, const void* K, const void* V,
                                const uint8_t* d_mask, const int32_t* q_idx, const int32_t* n_routed,
                                const int32_t* prefix, void* O, void* S_save, void* A_c, float* lse_loc,
                                float* lse_glb, void* fwd_ws, size_t fwd_ws_bytes, void* stream, int pair_begin,
                                int pair_end, bool clear_status, int row_begin = 0, int row_end = 0x7fffffff);

l2a_status l2a_forward(const l2a_params* p, const void* Q, const void* K, const void* V, const uint8_t* d_mask,
                       const int32_t* q_idx, const int32_t* n_routed, const int32_t* prefix, void* O, void* S_save,
                       void* A_c, float* lse_loc, float* lse_glb, void* fwd_ws, size_t fwd_ws_bytes, void* stream) {
  return forward_range(p, Q, K, V, d_mask, q_idx, n_routed, prefix, O, S_save, A_c, lse_loc, lse_glb, fwd_ws,
                       fwd_ws_bytes, stream, 0, -1, true);
}

// Section 3.1: Global Attention with its own Q/K/V (its own projections of the local output).  Local phase on
// (Q, K, V), then the global phase of the routed rows on (Qg, Kg, Vg), added into O.
l2a_status l2a_forward_sets(const l2a_params* p, const void* Q, const void* K, const void* V, const void* Qg,
                            const void* Kg, const void* Vg, const uint8_t* d_mask, const int32_t* q_idx,
                            const int32_t* n_routed, const int32_t* prefix, void* O, void* S_save, void* A_c,
                            float* lse_loc, float* lse_glb, void* fwd_ws, size_t fwd_ws_bytes, void* stream) {
  if (!p) return L2A_ERR_INVALID_ARG;
  if (!Qg && !Kg && !Vg)
    return l2a_forward(p, Q, K, V, d_mask, q_idx, n_routed, prefix, O, S_save, A_c, lse_loc, lse_glb, fwd_ws, fwd_ws_bytes,
                       stream);
  if (!Qg || !Kg || !Vg) return L2A_ERR_INVALID_ARG;
  if (p->flags & (L2A_FLAG_SKIP_LOCAL | L2A_FLAG_SKIP_GLOBAL | L2A_FLAG_GLOBAL_PHASE)) return L2A_ERR_INVALID_ARG;
  l2a_params q = *p;
  q.flags = (p->flags & ~(L2A_FLAG_SHARED_WINDOW | L2A_FLAG_FORCE_ALL_GLOBAL)) | L2A_FLAG_SKIP_GLOBAL;
  l2a_status st = forward_range(&q, Q, K, V, d_mask, q_idx, n_routed, prefix, O, S_save, A_c, lse_loc, lse_glb, fwd_ws,
                                fwd_ws_bytes, stream, 0, -1, true);
  if (st != L2A_OK) return st;
  q.flags = (p->flags & ~L2A_FLAG_SHARED_WINDOW) | L2A_FLAG_GLOBAL_PHASE;
  return forward_range(&q, Qg, Kg, Vg, d_mask, q_idx, n_routed, prefix, O, S_save, A_c, lse_loc, lse_glb, fwd_ws,
                       fwd_ws_bytes, stream, 0, -1, false);
}

static l2a_status forward_range(const l2a_params* p, const void* Q, const void* K, const void* V,
                                const uint8_t* d_mask, const int32_t* q_idx, const int32_t* n_routed,
                                const int32_t* prefix, void* O, void* S_save, void* A_c, float* lse_loc,
                                float* lse_glb, void* fwd_ws, size_t fwd_ws_bytes, void* stream, int pair_begin,
                                int pair_end, bool clear_status, int row_begin, int row_end) {
  l2a_status st = check_params(p);
  if (st != L2A_OK) return st;
  const bool save = p->flags & L2A_FLAG_SAVE_FOR_BWD;
  const bool skip_local = p->flags & L2A_FLAG_SKIP_LOCAL;
  const bool skip_global = p->flags & L2A_FLAG_SKIP_GLOBAL;
  const bool force_all = p->flags & L2A_FLAG_FORCE_ALL_GLOBAL;
  const bool global_phase = p->flags & L2A_FLAG_GLOBAL_PHASE;   // O already holds S: add the global part only
  if (skip_local && skip_global) return L2A_ERR_INVALID_ARG;
  if (global_phase && (skip_local || skip_global)) return L2A_ERR_INVALID_ARG;
  if (force_all && (!save || skip_local || skip_global)) return L2A_ERR_INVALID_ARG;
  if (!Q || !K || !V || !O) return L2A_ERR_INVALID_ARG;
  if (!skip_global && (!d_mask || !q_idx || !n_routed || !prefix)) return L2A_ERR_INVALID_ARG;
  if (save && (!S_save || !A_c || !lse_loc || !lse_glb)) return L2A_ERR_INVALID_ARG;
  if (save && skip_local) return L2A_ERR_INVALID_ARG;
  // shared-projection fusion concerns the global part only (a local-phase call just has to store lse_loc)
  const bool shared = (p->flags & L2A_FLAG_SHARED_WINDOW) && !skip_global;
  if (shared && (skip_local || force_all || !lse_loc)) return L2A_ERR_INVALID_ARG;
  if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) || !aligned(S_save, 16) ||
      !aligned(A_c, 16) || !aligned(lse_loc, 4) || !aligned(lse_glb, 4))
    return L2A_ERR_INVALID_ARG;
  if (!ws_ok(fwd_ws, fwd_ws_bytes, fwd_ws_size(p))) return L2A_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(fwd_ws);
  int* status = reinterpret_cast<int*>(ws);
  bf16* Qc = reinterpret_cast<bf16*>(ws + kWsHeaderBytes);
  const int n_pairs = ceil_div(p->Lq, kRowsPerCta);
  const bool whole = pair_end < 0 || (pair_begin == 0 && pair_end == n_pairs);
  if (pair_end < 0) pair_end = n_pairs;
  if (pair_begin < 0 || pair_end > n_pairs || pair_begin > pair_end) return L2A_ERR_INVALID_ARG;
  if (!whole && !skip_global) return L2A_ERR_INVALID_ARG;
  const bool row_range = row_begin > 0 || row_end < p->Lq;
  if (row_range && (!global_phase || row_begin < 0 || row_begin > row_end)) return L2A_ERR_INVALID_ARG;
  if (row_end > p->Lq) row_end = p->Lq;
  if (clear_status && cudaMemsetAsync(ws, 0, kWsHeaderBytes, s) != cudaSuccess) return L2A_ERR_CUDA;

  CUtensorMap mapQ, mapK, mapV, mapQc;
  const RowStrides qs = resolve_strides(p->q_stride, p->Lq, p->Hq * p->D);
  const RowStrides ks = resolve_strides(p->k_stride, p->Lk, p->Hkv * p->D);
  const RowStrides vs = resolve_strides(p->v_stride, p->Lk, p->Hkv * p->D);
  const RowStrides os = resolve_strides(p->o_stride, p->Lq, p->Hq * p->D);
  const RowStrides dense_q = {(int64_t)p->Lq * p->Hq * p->D, (int64_t)p->Hq * p->D};
  if (!encode_rows_map(&mapQ, Q, p->B, p->Lq, p->Hq * p->D, kTileM, p->D, qs.b, qs.t) ||
      !encode_rows_map(&mapK, K, p->B, p->Lk, p->Hkv * p->D, kTileN, p->D, ks.b, ks.t) ||
      !encode_rows_map(&mapV, V, p->B, p->Lk, p->Hkv * p->D, kTileN, p->D, vs.b, vs.t) ||
      !encode_rows_map(&mapQc, Qc, p->B, p->Lq, p->Hq * p->D, kTileM, p->D))
    return L2A_ERR_CUDA;

  FwdArgs a;
  a.B = p->B; a.Lq = p->Lq; a.Lk = p->Lk; a.Hq = p->Hq; a.Hkv = p->Hkv; a.D = p->D;
  a.window = p->window < (1 << 30) ? p->window : (1 << 30);   // any window >= Lk is the same; keeps W + 1 in range
  a.q_pos_offset = p->q_pos_offset;
  a.scale_log2 = scale_of(p) * 1.4426950408889634f;
  a.q_idx = q_idx;
  a.n_routed = n_routed;
  a.status = status;
  a.all_rows = 0;
  a.combine_mask = nullptr;
  a.pair_begin = 0;
  a.pair_end = n_pairs;
  a.row_begin = row_range ? row_begin : 0;
  a.row_end = row_range ? row_end : 0x7fffffff;
  a.shared_window = 0;
  a.lse_loc = nullptr;
  a.seq_bounds = p->seq_bounds;

  PhaseEvents& pe = phase_events();
  struct ClearOnExit { PhaseEvents& p; ~ClearOnExit() { p.clear(); } } clear_on_exit{pe};
  pe.mark(s);
  if (!skip_global && !force_all) {
    // consolidate routed query rows (Algorithm 1, step 1); independent of the local pass
    if (launch_gather_rows(static_cast<const bf16*>(Q), Qc, q_idx, n_routed, p->B, p->Lq, p->Hq * p->D, s,
                           row_range ? prefix : nullptr, row_begin, row_end, qs, status) != cudaSuccess)
      return L2A_ERR_CUDA;
  }
  pe.mark(s);
  if (!skip_local && !global_phase) {
    a.global_mode = 0;
    a.accumulate_into_out2 = 0;
    a.out = static_cast<bf16*>(save ? S_save : O);
    a.out2 = save ? static_cast<bf16*>(O) : nullptr;
    a.out_st = save ? dense_q : os;
    a.out2_st = os;
    a.lse = lse_loc;
    a.pair_begin = pair_begin;
    a.pair_end = pair_end;
    if (launch_attn_fwd(a, mapQ, mapK, mapV, s) != cudaSuccess) return L2A_ERR_CUDA;
    a.pair_begin = 0;
    a.pair_end = n_pairs;
  } else if (skip_local) {
    // Algorithm 1: O starts at zero (row by row when O is strided)
    for (int b = 0; b < p->B; ++b)
      if (cudaMemset2DAsync(static_cast<bf16*>(O) + b * os.b, (size_t)os.t * sizeof(bf16), 0,
                            (size_t)p->Hq * p->D * sizeof(bf16), p->Lq, s) != cudaSuccess)
        return L2A_ERR_CUDA;
  }
  pe.mark(s);
  if (!skip_global) {
    a.global_mode = 1;
    a.accumulate_into_out2 = skip_local ? 0 : 1;
    a.out = static_cast<bf16*>(A_c);
    a.out2 = static_cast<bf16*>(O);
    a.out_st = dense_q;
    a.out2_st = os;
    a.lse = lse_glb;
    a.shared_window = shared ? 1 : 0;
    a.lse_loc = lse_loc;
    if (force_all) {
      // Global Attention for every token (Section 3.3): same kernel over all rows in place; a_t is stored for
      // every row, and still only enters O where d_t = 1
      a.all_rows = 1;
      a.combine_mask = d_mask;
    }
    if (launch_attn_fwd(a, force_all ? mapQ : mapQc, mapK, mapV, s) != cudaSuccess) return L2A_ERR_CUDA;
  }
  pe.mark(s);
  return L2A_OK;
}

l2a_status l2a_router_logits(const l2a_params* p, const void* S, const float* w, float bias, float* logits,
                             float* sum_sq, void* stream) {
  l2a_status st = check_params(p);
  if (st != L2A_OK) return st;
  if (!S || !w || !logits) return L2A_ERR_INVALID_ARG;
  if (!aligned(S, 16) || !aligned(w, 16) || !aligned(logits, 4)) return L2A_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (sum_sq && cudaMemsetAsync(sum_sq, 0, sizeof(float) * p->B, s) != cudaSuccess) return L2A_ERR_CUDA;
  return launch_router_logits(static_cast<const bf16*>(S), w, bias, logits, sum_sq, p->B, p->Lq, p->Hq * p->D, s) ==
                 cudaSuccess
             ? L2A_OK
             : L2A_ERR_CUDA;
}

l2a_status l2a_router_backward(const l2a_params* p, const void* S, const float* w, const float* logits,
                               const float* dgate, float reg_coeff, const void* dO, float* dz, float* dw, float* dbias,
                               void* dS_loc, void* stream) {
  l2a_status st = check_params(p);
  if (st != L2A_OK) return st;
  if (!S || !w || !logits) return L2A_ERR_INVALID_ARG;
  if ((dO == nullptr) != (dS_loc == nullptr)) return L2A_ERR_INVALID_ARG;   // the combined gradient needs both
  if (dO != nullptr && !is_dense(p->o_stride, p->Lq, p->Hq * p->D)) return L2A_ERR_UNSUPPORTED;
  if (!aligned(S, 16) || !aligned(w, 16) || !aligned(dO, 16) || !aligned(dS_loc, 16) || !aligned(logits, 4) ||
      !aligned(dgate, 4) || !aligned(dz, 4) || !aligned(dw, 4) || !aligned(dbias, 4))
    return L2A_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dw && cudaMemsetAsync(dw, 0, sizeof(float) * p->Hq * p->D, s) != cudaSuccess) return L2A_ERR_CUDA;
  if (dbias && cudaMemsetAsync(dbias, 0, sizeof(float), s) != cudaSuccess) return L2A_ERR_CUDA;
  return launch_router_backward(static_cast<const bf16*>(S), w, logits, dgate, reg_coeff,
                                static_cast<const bf16*>(dO), dz, dw, dbias, static_cast<bf16*>(dS_loc), p->B, p->Lq,
                                p->Hq * p->D, s) == cudaSuccess
             ? L2A_OK
             : L2A_ERR_CUDA;
}

l2a_status l2a_forward_routed(const l2a_params* p, const void* Q, const void* K, const void* V, const float* router_w,
                              float router_bias, float logit_threshold, float* logits, float* sum_sq, uint8_t* d_mask,
                              int32_t* q_idx, int32_t* n_routed, int32_t* prefix, void* O, void* S_save, void* A_c,
                              float* lse_loc, float* lse_glb, void* route_ws, size_t route_ws_bytes, void* fwd_ws,
                              size_t fwd_ws_bytes, void* stream) {
  l2a_status st = check_params(p);
  if (st != L2A_OK) return st;
  if (p->flags & (L2A_FLAG_SKIP_LOCAL | L2A_FLAG_SKIP_GLOBAL | L2A_FLAG_GLOBAL_PHASE)) return L2A_ERR_INVALID_ARG;
  if (!router_w || !logits || !d_mask || !q_idx || !n_routed || !prefix) return L2A_ERR_INVALID_ARG;
  // every argument is checked before the first launch: the later stages would otherwise fail half-way
  if (!aligned(router_w, 16) || !aligned(logits, 4)) return L2A_ERR_INVALID_ARG;
  if (!ws_ok(route_ws, route_ws_bytes, route_ws_size(p)) || !ws_ok(fwd_ws, fwd_ws_bytes, fwd_ws_size(p)))
    return L2A_ERR_WORKSPACE;
  const bool save = p->flags & L2A_FLAG_SAVE_FOR_BWD;
  // Eq. 2: local attention for every token
  l2a_params ph = *p;
  ph.flags = (p->flags & ~L2A_FLAG_FORCE_ALL_GLOBAL) | L2A_FLAG_SKIP_GLOBAL;
  st = l2a_forward(&ph, Q, K, V, d_mask, q_idx, n_routed, prefix, O, S_save, A_c, lse_loc, lse_glb, fwd_ws,
                   fwd_ws_bytes, stream);
  if (st != L2A_OK) return st;
  // Eq. 3: router on the local output, threshold, compaction
  st = l2a_router_logits(p, save ? S_save : O, router_w, router_bias, logits, sum_sq, stream);
  if (st != L2A_OK) return st;
  st = l2a_route_compact(p, logits, L2A_ROUTER_LOGITS_F32, logit_threshold, d_mask, q_idx, n_routed, prefix, route_ws,
                         route_ws_bytes, stream);
  if (st != L2A_OK) return st;
  // Eq. 4 and 5: global attention of the routed tokens, added into O
  ph.flags = p->flags | L2A_FLAG_GLOBAL_PHASE;
  return l2a_forward(&ph, Q, K, V, d_mask, q_idx, n_routed, prefix, O, S_save, A_c, lse_loc, lse_glb, fwd_ws,
                     fwd_ws_bytes, stream);
}

l2a_status l2a_profile_next_call(void* const* events, int n_events) {
  if (n_events < 0 || n_events > 12 || (n_events > 0 && !events)) return L2A_ERR_INVALID_ARG;
  PhaseEvents& pe = phase_events();
  pe.clear();
  for (int i = 0; i < n_events; ++i) pe.ev[i] = static_cast<cudaEvent_t>(events[i]);
  pe.n = n_events;
  return L2A_OK;
}

// Helper streams and events of the host-buffer step, created once per host thread and device.
namespace {
struct StepAux {
  int device = -1;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, up = nullptr, fwd = nullptr, phase[11] = {}, down = nullptr, chunk[8] = {};
  // pipelined steps: kernels_done[k] / delivered[k] of the last two steps (k = step parity)
  cudaEvent_t kernels_done[2] = {}, delivered[2] = {};
  int n_async = 0;          // steps enqueued since the last wait
};
thread_local StepAux g_step_aux;
}  // namespace

static l2a_status step_host_impl(const l2a_params* p, const l2a_host_io* host, const l2a_device_io* dev,
                                 int router_kind, float logit_threshold, void* stream, bool async);

l2a_status l2a_step_host(const l2a_params* p, const l2a_host_io* host, const l2a_device_io* dev, int router_kind,
                         float logit_threshold, void* stream) {
  return step_host_impl(p, host, dev, router_kind, logit_threshold, stream, false);
}

l2a_status l2a_step_host_async(const l2a_params* p, const l2a_host_io* host, const l2a_device_io* dev,
                               int router_kind, float logit_threshold, void* stream) {
  return step_host_impl(p, host, dev, router_kind, logit_threshold, stream, true);
}

l2a_status l2a_step_host_wait(void* stream) {
  StepAux& aux = g_step_aux;
  aux.n_async = 0;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return L2A_ERR_CUDA;
  if (aux.device >= 0 && (cudaStreamSynchronize(aux.out) != cudaSuccess || cudaStreamSynchronize(aux.in) != cudaSuccess))
    return L2A_ERR_CUDA;
  return L2A_OK;
}

static l2a_status step_host_impl(const l2a_params* p, const l2a_host_io* host, const l2a_device_io* dev,
                                 int router_kind, float logit_threshold, void* stream, bool async) {
  l2a_status st = check_params(p);
  if (st != L2A_OK) return st;
  if (!host || !dev) return L2A_ERR_INVALID_ARG;
  if (p->seq_bounds) return L2A_ERR_UNSUPPORTED;   // the row-range pipeline assumes one sequence per batch entry
  const bool bwd = host->dO != nullptr;
  if (!host->Q || !host->K || !host->V || !host->router || !host->O || !dev->Q || !dev->K || !dev->V ||
      !dev->router || !dev->O)
    return L2A_ERR_INVALID_ARG;
  if (bwd && (!host->dQ || !host->dK || !host->dV || !dev->dO || !dev->dQ || !dev->dK || !dev->dV ||
              !(p->flags & L2A_FLAG_SAVE_FOR_BWD)))
    return L2A_ERR_INVALID_ARG;
  if (router_kind != L2A_ROUTER_MASK_U8 && router_kind != L2A_ROUTER_LOGITS_F32 &&
      router_kind != L2A_ROUTER_LOGITS_BF16)
    return L2A_ERR_INVALID_ARG;
  if (!is_dense(p->q_stride, p->Lq, p->Hq * p->D) || !is_dense(p->k_stride, p->Lk, p->Hkv * p->D) ||
      !is_dense(p->v_stride, p->Lk, p->Hkv * p->D) || !is_dense(p->o_stride, p->Lq, p->Hq * p->D))
    return L2A_ERR_UNSUPPORTED;     // host buffers and their device mirrors are dense
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t qb = (size_t)p->B * p->Lq * p->Hq * p->D * sizeof(bf16);
  const size_t kb = (size_t)p->B * p->Lk * p->Hkv * p->D * sizeof(bf16);
  const size_t rb = (size_t)p->B * p->Lq *
                    (router_kind == L2A_ROUTER_MASK_U8 ? 1 : router_kind == L2A_ROUTER_LOGITS_BF16 ? 2 : 4);
  // Two helper streams (created once per host thread and device) overlap the transfers with the kernels:
  // dO is uploaded while the forward runs, O is downloaded while the backward runs, dQ while the dK/dV kernel
  // runs (the backward computes dQ first for this reason); only dK and dV, the small results, leave after the
  // last kernel.  With pageable host memory the copies simply serialise.
  StepAux& aux = g_step_aux;
  int dev_id = 0;
  if (cudaGetDevice(&dev_id) != cudaSuccess) return L2A_ERR_CUDA;
  if (aux.device != dev_id) {
    if (cudaStreamCreateWithFlags(&aux.in, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&aux.out, cudaStreamNonBlocking) != cudaSuccess)
      return L2A_ERR_CUDA;
    cudaEvent_t* evs[] = {&aux.start, &aux.up, &aux.fwd, &aux.down, &aux.phase[0], &aux.phase[1], &aux.phase[2],
                          &aux.phase[3], &aux.phase[4], &aux.phase[5], &aux.phase[6], &aux.phase[7], &aux.phase[8],
                          &aux.phase[9], &aux.phase[10], &aux.chunk[0], &aux.chunk[1], &aux.chunk[2],
                          &aux.chunk[3], &aux.chunk[4], &aux.chunk[5], &aux.chunk[6], &aux.chunk[7],
                          &aux.kernels_done[0], &aux.kernels_done[1], &aux.delivered[0], &aux.delivered[1]};
    for (cudaEvent_t* e : evs)
      if (cudaEventCreateWithFlags(e, cudaEventDisableTiming) != cudaSuccess) return L2A_ERR_CUDA;
    aux.device = dev_id;
    aux.n_async = 0;
  }
#define L2A_TRY(x) do { if ((x) != cudaSuccess) return L2A_ERR_CUDA; } while (0)
  // Blocking step: the uploads start behind whatever the caller had queued on `stream` before this call.  Pipelined
  // step: they start behind the kernels of the step before the previous one (the last user of these device tensors),
  // and this step's kernels behind that step's downloads; the router input rides the upload stream as well.
  const int parity = aux.n_async & 1;
  if (!async && aux.n_async > 0) return L2A_ERR_INVALID_ARG;   // pipelined steps pending: l2a_step_host_wait first
  if (!async) {
    L2A_TRY(cudaEventRecord(aux.start, s));
    L2A_TRY(cudaMemcpyAsync(dev->router, host->router, rb, cudaMemcpyHostToDevice, s));
  } else {
    if (aux.n_async >= 2) {
      L2A_TRY(cudaStreamWaitEvent(aux.in, aux.kernels_done[parity], 0));
      L2A_TRY(cudaStreamWaitEvent(s, aux.delivered[parity], 0));
    }
    L2A_TRY(cudaMemcpyAsync(dev->router, host->router, rb, cudaMemcpyHostToDevice, aux.in));
    L2A_TRY(cudaEventRecord(aux.start, aux.in));
    L2A_TRY(cudaStreamWaitEvent(s, aux.start, 0));
  }
  l2a_params q = *p;
  if (!bwd) q.flags &= ~L2A_FLAG_SAVE_FOR_BWD;
  const bool need_lse_loc = bwd || (q.flags & L2A_FLAG_SHARED_WINDOW);   // the fusion reads it back in the forward
  const int n_pairs = ceil_div(p->Lq, kRowsPerCta);
  constexpr int kChunks = 8;
  // A pipelined step that follows another one has its transfers hidden behind that step's kernels: it uploads whole
  // tensors and runs one forward and one backward launch sequence instead of the row / key-block ranges, which exist
  // to start early and to drain early and cost a few percent of kernel time.
  const bool steady = async && aux.n_async > 0;
  const bool chunked = !steady && p->B == 1 && n_pairs >= 2 * kChunks &&
                       !(p->flags & (L2A_FLAG_SKIP_LOCAL | L2A_FLAG_SKIP_GLOBAL | L2A_FLAG_GLOBAL_PHASE));
  if (chunked) {
    // One sequence: K, V and Q go up in eight row ranges on the upload stream (attention is causal: the queries of a
    // range need no later keys); Local Attention and then the Global Attention of the routed rows of a range start
    // as soon as it has landed, so only the first range's copy is exposed.  Results equal a single l2a_forward call.
    if (!async) L2A_TRY(cudaStreamWaitEvent(aux.in, aux.start, 0));
    const size_t row_bytes = (size_t)p->Hq * p->D * sizeof(bf16), krow_bytes = (size_t)p->Hkv * p->D * sizeof(bf16);
    int pair_edge[kChunks + 1];
    for (int c = 0; c <= kChunks; ++c) pair_edge[c] = (int)((int64_t)n_pairs * c / kChunks);
    int64_t k_done = 0;   // key rows uploaded so far
    for (int c = 0; c < kChunks; ++c) {
      const int64_t r0 = (int64_t)pair_edge[c] * kRowsPerCta;
      int64_t r1 = (int64_t)pair_edge[c + 1] * kRowsPerCta;
      if (r1 > p->Lq) r1 = p->Lq;
      // the rows of this range see the keys up to position r1 - 1 + q_pos_offset (everything in the last range)
      int64_t k1 = c + 1 == kChunks ? p->Lk : r1 + p->q_pos_offset;
      if (k1 > p->Lk) k1 = p->Lk;
      if (k1 > k_done) {
        L2A_TRY(cudaMemcpyAsync(static_cast<uint8_t*>(dev->K) + k_done * krow_bytes,
                                static_cast<const uint8_t*>(host->K) + k_done * krow_bytes,
                                (size_t)(k1 - k_done) * krow_bytes, cudaMemcpyHostToDevice, aux.in));
        L2A_TRY(cudaMemcpyAsync(static_cast<uint8_t*>(dev->V) + k_done * krow_bytes,
                                static_cast<const uint8_t*>(host->V) + k_done * krow_bytes,
                                (size_t)(k1 - k_done) * krow_bytes, cudaMemcpyHostToDevice, aux.in));
        k_done = k1;
      }
      L2A_TRY(cudaMemcpyAsync(static_cast<uint8_t*>(dev->Q) + r0 * row_bytes,
                              static_cast<const uint8_t*>(host->Q) + r0 * row_bytes, (size_t)(r1 - r0) * row_bytes,
                              cudaMemcpyHostToDevice, aux.in));
      L2A_TRY(cudaEventRecord(aux.chunk[c], aux.in));
    }
    if (bwd) {
      L2A_TRY(cudaMemcpyAsync(dev->dO, host->dO, qb, cudaMemcpyHostToDevice, aux.in));
      L2A_TRY(cudaEventRecord(aux.up, aux.in));
    }
    st = l2a_route_compact(p, dev->router, router_kind, logit_threshold, dev->d_mask, dev->q_idx, dev->n_routed,
                           dev->prefix, dev->route_ws, dev->route_ws_bytes, stream);
    if (st != L2A_OK) return st;
    l2a_params ql = q, qg = q;
    ql.flags = (q.flags & ~L2A_FLAG_FORCE_ALL_GLOBAL) | L2A_FLAG_SKIP_GLOBAL;
    qg.flags |= L2A_FLAG_GLOBAL_PHASE;
    for (int c = 0; c < kChunks; ++c) {
      L2A_TRY(cudaStreamWaitEvent(s, aux.chunk[c], 0));
      st = forward_range(&ql, dev->Q, dev->K, dev->V, dev->d_mask, dev->q_idx, dev->n_routed, dev->prefix, dev->O,
                         bwd ? dev->S_save : nullptr, bwd ? dev->A_c : nullptr, need_lse_loc ? dev->lse_loc : nullptr,
                         bwd ? dev->lse_glb : nullptr, dev->fwd_ws, dev->fwd_ws_bytes, stream, pair_edge[c],
                         pair_edge[c + 1], c == 0);
      if (st != L2A_OK) return st;
      // Global Attention of the routed rows that have arrived so far: the compact groups whose last row lies in
      // this range (a group that straddles two ranges waits for the later one)
      const int r0 = pair_edge[c] * kRowsPerCta;
      const int r1 = c + 1 == kChunks ? p->Lq : pair_edge[c + 1] * kRowsPerCta;
      st = forward_range(&qg, dev->Q, dev->K, dev->V, dev->d_mask, dev->q_idx, dev->n_routed, dev->prefix, dev->O,
                         bwd ? dev->S_save : nullptr, bwd ? dev->A_c : nullptr, need_lse_loc ? dev->lse_loc : nullptr,
                         bwd ? dev->lse_glb : nullptr, dev->fwd_ws, dev->fwd_ws_bytes, stream, 0, -1, false, r0, r1);
      if (st != L2A_OK) return st;
    }
  } else {
    cudaStream_t us = async ? aux.in : s;
    L2A_TRY(cudaMemcpyAsync(dev->Q, host->Q, qb, cudaMemcpyHostToDevice, us));
    L2A_TRY(cudaMemcpyAsync(dev->K, host->K, kb, cudaMemcpyHostToDevice, us));
    L2A_TRY(cudaMemcpyAsync(dev->V, host->V, kb, cudaMemcpyHostToDevice, us));
    if (async) {
      L2A_TRY(cudaEventRecord(aux.chunk[0], aux.in));
      L2A_TRY(cudaStreamWaitEvent(s, aux.chunk[0], 0));
    }
    if (bwd) {   // dO rides the second stream, behind whatever the caller had queued before this call
      if (!async) L2A_TRY(cudaStreamWaitEvent(aux.in, aux.start, 0));
      L2A_TRY(cudaMemcpyAsync(dev->dO, host->dO, qb, cudaMemcpyHostToDevice, aux.in));
      L2A_TRY(cudaEventRecord(aux.up, aux.in));
    }
    st = l2a_route_compact(p, dev->router, router_kind, logit_threshold, dev->d_mask, dev->q_idx, dev->n_routed,
                           dev->prefix, dev->route_ws, dev->route_ws_bytes, stream);
    if (st != L2A_OK) return st;
    st = l2a_forward(&q, dev->Q, dev->K, dev->V, dev->d_mask, dev->q_idx, dev->n_routed, dev->prefix, dev->O,
                     bwd ? dev->S_save : nullptr, bwd ? dev->A_c : nullptr, need_lse_loc ? dev->lse_loc : nullptr,
                     bwd ? dev->lse_glb : nullptr, dev->fwd_ws, dev->fwd_ws_bytes, stream);
    if (st != L2A_OK) return st;
  }
  L2A_TRY(cudaEventRecord(aux.fwd, s));
  L2A_TRY(cudaStreamWaitEvent(aux.out, aux.fwd, 0));
  L2A_TRY(cudaMemcpyAsync(host->O, dev->O, qb, cudaMemcpyDeviceToHost, aux.out));
  if (bwd) {
    L2A_TRY(cudaStreamWaitEvent(s, aux.up, 0));
    // With eleven phase events the backward runs as four key-block ranges; boundary 4 + 2 r says that the gradients
    // range r completes (dK, dV of its keys, dQ of the rows that only see keys up to its end) are final: they leave on
    // the download stream while the next range is computed, the last range's after the last kernel.
    const int n_ev = steady ? 5 : 11;
    void* phase_events[11];
    for (int i = 0; i < 11; ++i) phase_events[i] = aux.phase[i];
    st = l2a_profile_next_call(phase_events, n_ev);
    if (st != L2A_OK) return st;
    st = l2a_backward(&q, dev->Q, dev->K, dev->V, dev->d_mask, dev->q_idx, dev->n_routed, dev->prefix, dev->dO,
                      dev->S_save, dev->A_c, dev->lse_loc, dev->lse_glb, dev->dQ, dev->dK, dev->dV, nullptr,
                      dev->bwd_ws, dev->bwd_ws_bytes, stream);
    if (st != L2A_OK) return st;
    int first[kMaxBwdRanges];
    const int n_kblocks = ceil_div(p->Lk, kTileN), n_tiles = ceil_div(p->Lq, kTileM);
    const int n_ranges = bwd_ranges(n_kblocks, n_ev, first);
    const size_t krow = (size_t)p->Hkv * p->D * sizeof(bf16), qrow = (size_t)p->Hq * p->D * sizeof(bf16);
    int64_t k_done = 0, q_done = 0;
    for (int r = 0; r < n_ranges; ++r) {
      const bool last = r + 1 == n_ranges;
      int64_t k_end = last ? p->Lk : (int64_t)first[r + 1] * kTileN;
      int64_t q_end = last ? p->Lq : (int64_t)dq_final_tiles(first[r + 1], p->q_pos_offset, n_tiles) * kTileM;
      if (k_end > p->Lk) k_end = p->Lk;
      if (q_end > p->Lq) q_end = p->Lq;
      cudaStream_t cs = (last && !async) ? s : aux.out;
      if (!last || async) L2A_TRY(cudaStreamWaitEvent(aux.out, aux.phase[4 + 2 * r], 0));
      for (int b = 0; b < p->B; ++b) {
        const size_t kbase = (size_t)b * p->Lk * krow, qbase = (size_t)b * p->Lq * qrow;
        if (q_end > q_done)
          L2A_TRY(cudaMemcpyAsync(static_cast<uint8_t*>(host->dQ) + qbase + q_done * qrow,
                                  static_cast<const uint8_t*>(dev->dQ) + qbase + q_done * qrow,
                                  (size_t)(q_end - q_done) * qrow, cudaMemcpyDeviceToHost, cs));
        if (k_end > k_done) {
          L2A_TRY(cudaMemcpyAsync(static_cast<uint8_t*>(host->dK) + kbase + k_done * krow,
                                  static_cast<const uint8_t*>(dev->dK) + kbase + k_done * krow,
                                  (size_t)(k_end - k_done) * krow, cudaMemcpyDeviceToHost, cs));
          L2A_TRY(cudaMemcpyAsync(static_cast<uint8_t*>(host->dV) + kbase + k_done * krow,
                                  static_cast<const uint8_t*>(dev->dV) + kbase + k_done * krow,
                                  (size_t)(k_end - k_done) * krow, cudaMemcpyDeviceToHost, cs));
        }
      }
      if (q_end > q_done) q_done = q_end;
      if (k_end > k_done) k_done = k_end;
    }
  }
  if (async) {
    // nothing on `stream` waits for the downloads: the next step's kernels follow this step's directly
    L2A_TRY(cudaEventRecord(aux.kernels_done[parity], s));
    L2A_TRY(cudaEventRecord(aux.delivered[parity], aux.out));
    ++aux.n_async;
    return L2A_OK;
  }
  L2A_TRY(cudaEventRecord(aux.down, aux.out));
  L2A_TRY(cudaStreamWaitEvent(s, aux.down, 0));   // the caller's stream ends the step with every result delivered
  L2A_TRY(cudaStreamSynchronize(s));
#undef L2A_TRY
  return L2A_OK;
}

}  // extern "C"
