// Flat-shard gather/scatter: pure byte movement between the padded 1-D shard buffer and whole
// row-major matrices (the unpack after a fused gather and the pack before the relay broadcast,
// Section 6.4 steps 1 and 3).  HBM-bound; 16-byte vector loads/stores whenever both sides of a
// work item can be brought to a common 16-byte phase, element-wise otherwise.
#include "internal.h"

namespace muon {

// One block per work item (<= kCopyChunk elements).  `scatter` selects the direction.
template <int ES>
__global__ void __launch_bounds__(256) copy_items_kernel(const CopyItem* __restrict__ items, char* __restrict__ flat,
                                                         void* const* __restrict__ mats, int scatter) {
  const CopyItem it = items[blockIdx.x];
  if (!mats[it.matrix]) return;                    // block-uniform: a matrix the caller left out (subset calls)
  char* fptr = flat + it.flat_offset * ES;
  char* mptr = static_cast<char*>(mats[it.matrix]) + it.elem_begin * ES;
  const char* src = scatter ? mptr : fptr;
  char* dst = scatter ? fptr : mptr;
  const int64_t bytes = int64_t(it.count) * ES;
  const unsigned sa = unsigned(reinterpret_cast<uintptr_t>(src) & 15u);
  const unsigned da = unsigned(reinterpret_cast<uintptr_t>(dst) & 15u);
  using elem_t = typename std::conditional<ES == 2, uint16_t, uint32_t>::type;
  if (sa != da) {  // no common phase: move element by element (still coalesced)
    const elem_t* s = reinterpret_cast<const elem_t*>(src);
    elem_t* d = reinterpret_cast<elem_t*>(dst);
    for (int i = threadIdx.x; i < it.count; i += blockDim.x) d[i] = s[i];
    return;
  }
  int64_t head = sa ? (16 - sa) : 0;
  if (head > bytes) head = bytes;
  const int64_t body = (bytes - head) / 16;       // number of 16-byte vectors
  const int64_t tail_begin = head + body * 16;
  {  // ragged head and tail, element-wise
    const int head_e = int(head / ES), tail_e = int((bytes - tail_begin) / ES);
    const elem_t* s = reinterpret_cast<const elem_t*>(src);
    elem_t* d = reinterpret_cast<elem_t*>(dst);
    if (int(threadIdx.x) < head_e) d[threadIdx.x] = s[threadIdx.x];
    if (int(threadIdx.x) < tail_e) {
      const int64_t e = tail_begin / ES + threadIdx.x;
      d[e] = s[e];
    }
  }
  const uint4* s4 = reinterpret_cast<const uint4*>(src + head);
  uint4* d4 = reinterpret_cast<uint4*>(dst + head);
  int64_t i = threadIdx.x;
  // four independent 16-byte loads in flight per thread before the stores
  for (; i + 3 * 256 < body; i += 4 * 256) {
    const uint4 v0 = __ldcs(s4 + i), v1 = __ldcs(s4 + i + 256), v2 = __ldcs(s4 + i + 512), v3 = __ldcs(s4 + i + 768);
    __stcs(d4 + i, v0);
    __stcs(d4 + i + 256, v1);
    __stcs(d4 + i + 512, v2);
    __stcs(d4 + i + 768, v3);
  }
  for (; i < body; i += 256) __stcs(d4 + i, __ldcs(s4 + i));
}

// ---------------------------------------------------------------------------------------------------------------
// Shard-local halves of the owner-sharded step (Section 6.4): what a rank does to the shard it holds, without ever
// seeing a whole matrix.  Both kernels walk the copy items of ONE shard (one block per item of <= kCopyChunk
// elements) and address the rank's local buffers relative to the shard's first element; padding is never touched.
//   momentum (step 1, before the fused gather): M <- mu*M + G, staged = cast(G + mu*M) (Nesterov) or cast(M);
//            the staged shard is what the gather sends ("packs a whole batch of momentum shards ... bf16").
//   apply    (step 4, after the relay broadcast): W <- W(1 - lr*wd) - lr * 0.2 sqrt(max(m,n)) * O, where O is the
//            owner's whole-matrix update and the rank extracts its own slice of it on the fly.
// The arithmetic is written with explicit roundings, the same as in the fused whole-matrix kernels, so that a
// step assembled from these halves is bit-identical to muon_step_batched.
// ---------------------------------------------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float ld_as_float(const T* p);
template <> __device__ __forceinline__ float ld_as_float<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld_as_float<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ T st_from_float(float v);
template <> __device__ __forceinline__ float st_from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 st_from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename GT, typename XT>
__global__ void __launch_bounds__(256) shard_momentum_kernel(const CopyItem* __restrict__ items, int64_t shard_base,
                                                             const GT* __restrict__ g, float* __restrict__ m,
                                                             XT* __restrict__ staged, float mu, int nesterov) {
  const CopyItem it = items[blockIdx.x];
  const int64_t off = it.flat_offset - shard_base;
  const GT* gp = g + off;
  float* mp = m + off;
  XT* sp = staged + off;
  for (int i = threadIdx.x; i < it.count; i += blockDim.x) {
    const float gv = ld_as_float<GT>(gp + i);
    const float mv = __fmaf_rn(mu, mp[i], gv);
    mp[i] = mv;
    sp[i] = st_from_float<XT>(nesterov ? __fmaf_rn(mu, mv, gv) : mv);
  }
}

template <typename XT>
__global__ void __launch_bounds__(256) shard_apply_kernel(const CopyItem* __restrict__ items, int64_t shard_base,
                                                          float* __restrict__ w, const void* const* __restrict__ updates,
                                                          const float* __restrict__ scales, float lr, float decay) {
  const CopyItem it = items[blockIdx.x];
  const XT* o = static_cast<const XT*>(updates[it.matrix]);
  if (!o) return;                                   // block-uniform: a matrix without an update is left alone
  o += it.elem_begin;
  float* wp = w + (it.flat_offset - shard_base);
  const float step = lr * scales[it.matrix];
  for (int i = threadIdx.x; i < it.count; i += blockDim.x)
    wp[i] = __fmaf_rn(-step, ld_as_float<XT>(o + i), __fmul_rn(wp[i], decay));
}

int launch_shard_momentum(const CopyItem* items, int64_t num_items, int64_t shard_base, const void* g, void* m, void* staged,
                          float mu, int nesterov, int grad_dtype, int ns_precision, cudaStream_t st) {
  if (num_items == 0) return 0;
  if (num_items > 0x7fffffffLL) return MUON_ERR_UNSUPPORTED;
  const unsigned n = unsigned(num_items);
  const bool gbf = grad_dtype == MUON_DTYPE_BF16, xbf = ns_precision == MUON_NS_BF16;
  float* mf = static_cast<float*>(m);
  if (gbf && xbf)
    shard_momentum_kernel<__nv_bfloat16, __nv_bfloat16><<<n, 256, 0, st>>>(items, shard_base, static_cast<const __nv_bfloat16*>(g), mf,
                                                                           static_cast<__nv_bfloat16*>(staged), mu, nesterov);
  else if (gbf)
    shard_momentum_kernel<__nv_bfloat16, float><<<n, 256, 0, st>>>(items, shard_base, static_cast<const __nv_bfloat16*>(g), mf,
                                                                   static_cast<float*>(staged), mu, nesterov);
  else if (xbf)
    shard_momentum_kernel<float, __nv_bfloat16><<<n, 256, 0, st>>>(items, shard_base, static_cast<const float*>(g), mf,
                                                                   static_cast<__nv_bfloat16*>(staged), mu, nesterov);
  else
    shard_momentum_kernel<float, float><<<n, 256, 0, st>>>(items, shard_base, static_cast<const float*>(g), mf,
                                                           static_cast<float*>(staged), mu, nesterov);
  return cudaGetLastError() == cudaSuccess ? 1 : MUON_ERR_CUDA;
}

int launch_shard_apply(const CopyItem* items, int64_t num_items, int64_t shard_base, void* w, const void* const* d_updates,
                       const float* d_scales, float lr, float decay, int ns_precision, cudaStream_t st) {
  if (num_items == 0) return 0;
  if (num_items > 0x7fffffffLL) return MUON_ERR_UNSUPPORTED;
  const unsigned n = unsigned(num_items);
  if (ns_precision == MUON_NS_BF16)
    shard_apply_kernel<__nv_bfloat16><<<n, 256, 0, st>>>(items, shard_base, static_cast<float*>(w), d_updates, d_scales, lr, decay);
  else
    shard_apply_kernel<float><<<n, 256, 0, st>>>(items, shard_base, static_cast<float*>(w), d_updates, d_scales, lr, decay);
  return cudaGetLastError() == cudaSuccess ? 1 : MUON_ERR_CUDA;
}

int launch_copy(const CopyItem* items, int64_t num_items, void* flat, void* const* d_mats, int elem_size, bool scatter,
                cudaStream_t st) {
  if (num_items == 0) return 0;
  if (num_items > 0x7fffffffLL) return MUON_ERR_UNSUPPORTED;
  if (elem_size == 2)
    copy_items_kernel<2><<<unsigned(num_items), 256, 0, st>>>(items, static_cast<char*>(flat), d_mats, scatter ? 1 : 0);
  else
    copy_items_kernel<4><<<unsigned(num_items), 256, 0, st>>>(items, static_cast<char*>(flat), d_mats, scatter ? 1 : 0);
  return cudaGetLastError() == cudaSuccess ? 1 : MUON_ERR_CUDA;
}

}  // namespace muon
