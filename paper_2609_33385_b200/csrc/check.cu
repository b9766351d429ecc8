// Self-check of a step (no counterpart in the paper; a stand-in for a memory checker on systems
// where none can be run).  Two kernels, both off unless OLED_OPT_SELF_CHECK is set:
//   * after the permutation: the routing and permutation invariants every later kernel relies on
//     for its addressing - expert ids in range and distinct per token, offsets the exclusive scan
//     of the counts, perm a bijection with pos its inverse, every sorted row inside the range of
//     the expert its assignment was routed to, rows of an expert in ascending assignment order;
//   * after the combine: the guard words behind the step's scratch buffers are intact.
// A violation sets a flag (and the smallest offending index) in the context's status block; the
// next synchronising call returns OLED_ERR_SELF_CHECK.  Nothing is skipped or repaired.
#include <algorithm>

#include "kernels.h"

namespace oled {
namespace {

__device__ __forceinline__ void report(uint32_t* status, uint32_t flag, int index) {
  atomicOr(&status[kStatusCheckFlags], flag);
  atomicMin(reinterpret_cast<int*>(&status[kStatusCheckIndex]), index);
}

__global__ void __launch_bounds__(256)
self_check_kernel(const int32_t* __restrict__ ids, const int32_t* __restrict__ counts,
                  const int32_t* __restrict__ offsets, const int32_t* __restrict__ perm,
                  const int32_t* __restrict__ pos, int T, int E, int K, uint32_t* __restrict__ status) {
  const int n = T * K;
  const int tid = blockIdx.x * blockDim.x + threadIdx.x, step = gridDim.x * blockDim.x;
  // offsets: exclusive scan of the counts
  for (int e = tid; e < E; e += step) {
    if (offsets[e + 1] - offsets[e] != counts[e] || counts[e] < 0) report(status, OLED_CHECK_OFFSETS, e);
    if (e == 0 && offsets[0] != 0) report(status, OLED_CHECK_OFFSETS, 0);
    if (e == E - 1 && offsets[E] != n) report(status, OLED_CHECK_OFFSETS, E);
  }
  // ids: in range, distinct within a token
  for (int t = tid; t < T; t += step) {
    for (int j = 0; j < K; ++j) {
      const int id = ids[t * K + j];
      if (id < 0 || id >= E) report(status, OLED_CHECK_ID_RANGE, t * K + j);
      for (int j2 = 0; j2 < j; ++j2)
        if (ids[t * K + j2] == id) report(status, OLED_CHECK_ID_DUPLICATE, t * K + j);
    }
  }
  // sorted rows: perm in range, pos its inverse, the row inside its expert's range, stable order
  for (int r = tid; r < n; r += step) {
    const int a = perm[r];
    if (a < 0 || a >= n) {
      report(status, OLED_CHECK_PERM_RANGE, r);
      continue;
    }
    if (pos[a] != r) report(status, OLED_CHECK_INVERSE, r);
    const int id = ids[a];
    if (id >= 0 && id < E) {
      if (r < offsets[id] || r >= offsets[id + 1]) report(status, OLED_CHECK_ROW_EXPERT, r);
      else if (r > offsets[id] && perm[r - 1] >= a) report(status, OLED_CHECK_ORDER, r);
    }
  }
}

__global__ void guard_check_kernel(GuardList guards, uint32_t* __restrict__ status) {
  const int b = blockIdx.x;
  if (b >= guards.n) return;
  const uint32_t* g = guards.words[b];
  if (threadIdx.x < kGuardWords && g[threadIdx.x] != kGuardPattern) atomicOr(&status[kStatusGuardMask], 1u << b);
}

__global__ void guard_fill_kernel(GuardList guards) {
  const int b = blockIdx.x;
  if (b < guards.n && threadIdx.x < kGuardWords) guards.words[b][threadIdx.x] = kGuardPattern;
}

// Test aid: exchanges the first two entries of the sorted order (both stay in range, so every later
// kernel still addresses valid rows; the step's output is wrong and the self-check must say so).
__global__ void corrupt_perm_kernel(int32_t* perm, int n) {
  if (n >= 2 && threadIdx.x == 0 && blockIdx.x == 0) {
    const int a = perm[0];
    perm[0] = perm[1];
    perm[1] = a;
  }
}

}  // namespace

void launch_self_check(cudaStream_t st, const int32_t* ids, const int32_t* counts, const int32_t* offsets,
                       const int32_t* perm, const int32_t* pos, int T, int E, int K, uint32_t* status) {
  const int n = T * K;
  const int blocks = std::max(1, std::min(148, (std::max(n, E) + 255) / 256));
  self_check_kernel<<<blocks, 256, 0, st>>>(ids, counts, offsets, perm, pos, T, E, K, status);
}

void launch_guard_check(cudaStream_t st, const GuardList& guards, uint32_t* status) {
  if (guards.n > 0) guard_check_kernel<<<guards.n, 32, 0, st>>>(guards, status);
}

void launch_guard_fill(cudaStream_t st, const GuardList& guards) {
  if (guards.n > 0) guard_fill_kernel<<<guards.n, 32, 0, st>>>(guards);
}

void launch_corrupt_perm(cudaStream_t st, int32_t* perm, int n) { corrupt_perm_kernel<<<1, 32, 0, st>>>(perm, n); }

}  // namespace oled
