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
