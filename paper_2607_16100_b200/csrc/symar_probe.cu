// Speed-of-light probes (paper Sec. VI): the pieces of the latency lower bound,
// measured on the device the collective runs on.
//
//   L_L2_RTT        one __threadfence() with one store outstanding: the SM must
//                   wait until the store has reached L2, the point of coherence;
//   flag round trip one 4-byte value bounced between two CTAs on two SMs through
//                   L2 -- the one-GPU counterpart of the paper's two-GPU
//                   ping-pong, L_pingpong = 2 L_L2_RTT + 2 L_remote_store;
//   launch floor    an empty kernel of the same grid and block as the collective.
//
// Every spin is bounded; a probe that gives up returns SYMAR_ERR_TIMEOUT.
#include <cuda_runtime.h>

#include "symar.h"

namespace {

__device__ __forceinline__ unsigned long long timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ unsigned ld_relaxed(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed(unsigned *p, unsigned v)
{
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

__global__ void empty_kernel() {}
__global__ void empty_pdl_kernel()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");
}

// out[0] = elapsed ns over `iters` store+fence pairs
__global__ void fence_kernel(unsigned *scratch, int iters, unsigned long long *out)
{
    unsigned long long t0 = timer_ns();
    for (int i = 0; i < iters; ++i) {
        st_relaxed(scratch, (unsigned)i);
        __threadfence();
    }
    unsigned long long t1 = timer_ns();
    out[0] = t1 - t0;
}

constexpr unsigned kSpinLimit = 1u << 22;   // polls; far above any real round trip

// flags[0] is written by the first block and watched by its partner; flags[32] the reverse
// (separate 128-byte lines).  out[0] = ns, out[1] = 1 on timeout, out[2..3] = SM ids.
__global__ void pingpong_kernel(unsigned *flags, int iters, unsigned long long *out, int first, int partner)
{
    // blocks other than `first` and `partner` only fill the SMs in between
    if ((int)blockIdx.x != first && (int)blockIdx.x != partner) return;
    const bool starts = (int)blockIdx.x == first;
    unsigned smid;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    unsigned *mine   = flags + (starts ? 0 : 32);
    unsigned *theirs = flags + (starts ? 32 : 0);
    out[2 + (starts ? 0 : 1)] = smid;
    bool dead = false;
    unsigned long long t0 = 0;
    if (starts) {
        // one untimed exchange first, so that both blocks are known to be running
        for (int i = 1; i <= iters + 1 && !dead; ++i) {
            if (i == 2) t0 = timer_ns();
            st_relaxed(mine, (unsigned)i);
            unsigned n = 0;
            while (ld_relaxed(theirs) != (unsigned)i)
                if (++n > kSpinLimit) { dead = true; break; }
        }
        out[0] = timer_ns() - t0;
    } else {
        for (int i = 1; i <= iters + 1 && !dead; ++i) {
            unsigned n = 0;
            while (ld_relaxed(theirs) != (unsigned)i)
                if (++n > kSpinLimit) { dead = true; break; }
            st_relaxed(mine, (unsigned)i);
        }
    }
    if (dead) out[1] = 1;
}

// The barrier the method removes (paper Sec. III-B): every rank signals every peer and waits
// for every peer, `iters` times in a row.  One CTA per rank, lane q of warp 0 talks to peer q;
// flags[rank][peer] counts the barriers that `peer` has entered.  mode 0: relaxed signals (the
// paper's measurement); mode 1: release signals + acquire polls (a barrier that orders memory).
// out[0] = ns over all iterations as seen by rank 0, out[1] = 1 on timeout.
__global__ void barrier_kernel(unsigned *flags, int iters, int mode, unsigned long long *out)
{
    const int P = gridDim.x, r = blockIdx.x;
    const unsigned lane = threadIdx.x;
    if (lane >= 32) return;
    unsigned *sig        = flags + (size_t)(lane < (unsigned)P ? lane : 0) * 32 + r;    // my word in peer `lane`'s row
    const unsigned *mine = flags + (size_t)r * 32 + (lane < (unsigned)P ? lane : 0);   // peer `lane`'s word in my row
    bool dead = false;
    unsigned long long t0 = 0;
    for (int i = 1; i <= iters + 1 && !dead; ++i) {
        if (i == 2) t0 = timer_ns();                    // the first barrier only lines the CTAs up
        if (lane < (unsigned)P) {
            if (mode == 1) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(sig) : "memory");
            else asm volatile("red.relaxed.gpu.global.add.u32 [%0], 1;" ::"l"(sig) : "memory");
        }
        unsigned n = 0;
        for (;;) {
            unsigned f;
            if (mode == 1) asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(f) : "l"(mine) : "memory");
            else f = ld_relaxed(mine);
            if (__ballot_sync(0xffffffffu, lane < (unsigned)P && (int)(f - (unsigned)i) < 0) == 0) break;
            if (++n > kSpinLimit) { dead = true; break; }
        }
    }
    if (r == 0 && lane == 0) {
        out[0] = timer_ns() - t0;
        out[1] = dead ? 1 : 0;
    } else if (dead && lane == 0) {
        out[1] = 1;
    }
}

int sync_and_fetch(unsigned long long *dev, unsigned long long *host, int n)
{
    if (cudaDeviceSynchronize() != cudaSuccess) return SYMAR_ERR_CUDA;
    if (cudaMemcpy(host, dev, n * sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess)
        return SYMAR_ERR_CUDA;
    return SYMAR_OK;
}

}  // namespace

extern "C" {

int symar_probe_empty(int grid_x, int grid_y, int block, void *cuda_stream)
{
    if (grid_x < 1 || grid_y < 1 || block < 1 || block > 1024) return SYMAR_ERR_INVAL;
    empty_kernel<<<dim3(grid_x, grid_y, 1), block, 0, (cudaStream_t)cuda_stream>>>();
    return cudaGetLastError() == cudaSuccess ? SYMAR_OK : SYMAR_ERR_CUDA;
}

int symar_probe_empty_pdl(int grid_x, int grid_y, int block, void *cuda_stream)
{
    if (grid_x < 1 || grid_y < 1 || block < 1 || block > 1024) return SYMAR_ERR_INVAL;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim  = dim3(grid_x, grid_y, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.stream   = (cudaStream_t)cuda_stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs    = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, empty_pdl_kernel) == cudaSuccess ? SYMAR_OK : SYMAR_ERR_CUDA;
}

int symar_probe_empty_cluster(int grid_x, int grid_y, int block, void *cuda_stream)
{
    if (grid_x < 1 || grid_y < 2 || grid_y > 8 || block < 1 || block > 1024) return SYMAR_ERR_INVAL;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim  = dim3(grid_x, grid_y, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.stream   = (cudaStream_t)cuda_stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id               = cudaLaunchAttributeClusterDimension;     // the grid_y CTAs of a column as one cluster
    attr[1].val.clusterDim.x = 1;
    attr[1].val.clusterDim.y = (unsigned)grid_y;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs    = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, empty_pdl_kernel) == cudaSuccess ? SYMAR_OK : SYMAR_ERR_CUDA;
}

int symar_probe_fence(int iterations, double *host_ns_per_fence)
{
    if (iterations < 1 || !host_ns_per_fence) return SYMAR_ERR_INVAL;
    unsigned char *buf = nullptr;
    if (cudaMalloc(&buf, 512) != cudaSuccess) return SYMAR_ERR_NOMEM;
    cudaMemset(buf, 0, 512);
    unsigned long long h[4] = {0, 0, 0, 0};
    fence_kernel<<<1, 1>>>((unsigned *)buf, 16, (unsigned long long *)(buf + 256));   // warm
    fence_kernel<<<1, 1>>>((unsigned *)buf, iterations, (unsigned long long *)(buf + 256));
    int rc = sync_and_fetch((unsigned long long *)(buf + 256), h, 1);
    cudaFree(buf);
    if (rc != SYMAR_OK) return rc;
    *host_ns_per_fence = (double)h[0] / iterations;
    return SYMAR_OK;
}

int symar_probe_barrier(int ranks, int iterations, int ordered, double *host_ns_per_barrier)
{
    if (ranks < 2 || ranks > 32 || iterations < 1 || !host_ns_per_barrier) return SYMAR_ERR_INVAL;
    unsigned char *buf = nullptr;
    const size_t flag_bytes = 32 * 32 * sizeof(unsigned);                   // one 128-byte row per rank
    if (cudaMalloc(&buf, flag_bytes + 256) != cudaSuccess) return SYMAR_ERR_NOMEM;
    cudaMemset(buf, 0, flag_bytes + 256);
    unsigned long long h[2] = {0, 0};
    barrier_kernel<<<ranks, 32>>>((unsigned *)buf, iterations, ordered ? 1 : 0, (unsigned long long *)(buf + flag_bytes));
    int rc = sync_and_fetch((unsigned long long *)(buf + flag_bytes), h, 2);
    cudaFree(buf);
    if (rc != SYMAR_OK) return rc;
    if (h[1] != 0) return SYMAR_ERR_TIMEOUT;
    *host_ns_per_barrier = (double)h[0] / iterations;
    return SYMAR_OK;
}

int symar_probe_pingpong_blocks(int iterations, int first_block, int partner_block, int grid_blocks,
                                double *host_ns_per_round_trip, int *host_smids)
{
    if (iterations < 1 || grid_blocks < 2 || grid_blocks > 1024 || first_block < 0 || partner_block < 0 ||
        first_block >= grid_blocks || partner_block >= grid_blocks || first_block == partner_block ||
        !host_ns_per_round_trip)
        return SYMAR_ERR_INVAL;
    unsigned char *buf = nullptr;
    if (cudaMalloc(&buf, 1024) != cudaSuccess) return SYMAR_ERR_NOMEM;
    cudaMemset(buf, 0, 1024);
    unsigned long long h[4] = {0, 0, 0, 0};
    pingpong_kernel<<<grid_blocks, 1>>>((unsigned *)buf, iterations, (unsigned long long *)(buf + 512), first_block,
                                        partner_block);
    int rc = sync_and_fetch((unsigned long long *)(buf + 512), h, 4);
    cudaFree(buf);
    if (rc != SYMAR_OK) return rc;
    if (h[1] != 0) return SYMAR_ERR_TIMEOUT;
    if (host_smids) {
        host_smids[0] = (int)h[2];
        host_smids[1] = (int)h[3];
    }
    if (h[2] == h[3]) return SYMAR_ERR_UNSUPPORTED;   // both blocks landed on one SM: not an L2 round trip
    *host_ns_per_round_trip = (double)h[0] / iterations;
    return SYMAR_OK;
}

int symar_probe_pingpong_pair(int iterations, int partner_block, double *host_ns_per_round_trip,
                              int *host_smids)
{
    if (partner_block < 1 || partner_block > 1023) return SYMAR_ERR_INVAL;
    return symar_probe_pingpong_blocks(iterations, 0, partner_block, partner_block + 1, host_ns_per_round_trip,
                                       host_smids);
}

int symar_probe_pingpong(int iterations, double *host_ns_per_round_trip)
{
    return symar_probe_pingpong_pair(iterations, 1, host_ns_per_round_trip, nullptr);
}

}  // extern "C"
