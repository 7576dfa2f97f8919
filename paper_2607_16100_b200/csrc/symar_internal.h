// Declarations shared by the translation units of libsymar (host side).
#pragma once
#include <cuda_runtime.h>

#include "symar_layout.h"

namespace symar {

using KernelFn = void (*)(const KArgs);

// Kernel instantiation for (algorithm, element type, ranks); dbg selects the
// variant that honours the test hooks.  nullptr for unsupported combinations.
KernelFn kernel_for(int algo, int dtype, int P, bool dbg);

// LL for messages that one iteration covers with one unit of `words` (2 or 4) 32-bit words per thread.
KernelFn ll_small_kernel_for(int dtype, int P, int words, bool dbg);

// Two-shot kernel of the bandwidth regime (bulk asynchronous copies through
// shared memory); needs bulk_smem_bytes() of dynamic shared memory.
KernelFn bulk_kernel_for(int dtype, int P);

// Two-shot with atomic accumulation in the owner's scratch (symar_atomic.cu).
KernelFn atomic_kernel_for(int dtype, int P, bool dbg);

// grid = (ctas_per_rank, P), block = threads; returns the launch status.
cudaError_t launch_kernel(KernelFn fn, int P, int ctas_per_rank, int threads, size_t smem_bytes,
                          const KArgs &args, cudaStream_t stream, bool cluster = false);
int max_resident_clusters(KernelFn fn, int P, int threads, size_t smem_bytes);

// Variant bit common to all algorithms (host side only, never passed to a kernel): launch the P CTAs of
// a slot as one thread-block cluster.
constexpr unsigned kVarCluster = SYMAR_VARIANT_CLUSTER;

// Placement on the chip's two L2 halves (symar_place.cu): which half every SM sits on, and which half
// homes copy 0 of every flag / counter pair of a heap.  `scratch`: 3 * kPairBytes of device memory,
// 8 KiB-aligned, left zeroed.  *ok = false (and all-zero results) when the measurement is not clean.
cudaError_t place_measure_sms(unsigned char *scratch, int num_sms, int max_smem_optin, uint64_t sm_half[4], bool *ok);
cudaError_t place_measure_heap(char *seg0, size_t stride, int P, const Layout &L, const uint64_t sm_half[4],
                               unsigned char *scratch, uint64_t *home, bool *ok);

// Checking build only (cudaErrorNotSupported otherwise): the kernel behind symar_check_selftest().
cudaError_t launch_check_selftest(const KArgs &args, cudaStream_t stream);

// Sibling collectives (symar_coll.cu): op = 0 ReduceScatter, 1 AllGather, 2 Broadcast, 3 Reduce.
cudaError_t launch_collective(int op, int dtype, int P, int ctas_per_rank, int threads, const KArgs &k,
                              uint64_t bytes, int root, int unit, cudaStream_t stream, bool cluster = false);
int collective_resident_clusters(int op, int dtype, int P, int threads);
int collective_resident(int op, int dtype, int P, int threads, int num_sms);

}  // namespace symar
