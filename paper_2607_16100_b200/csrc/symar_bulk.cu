// Two-shot AllReduce for the bandwidth regime (paper Sec. III-A.2: reduce-scatter,
// then all-gather), built on Blackwell's bulk asynchronous copy engine.
//
// Rank r owns the tiles g with g mod P == r (a tile is `tile_vecs` 16-byte
// vectors, 4 KiB by default).  CTA (r, c) walks its share of those tiles with a
// `stages`-deep pipeline:
//
//   load    one elected thread issues P bulk copies global -> shared (the tile
//           of every rank's input), completion counted in bytes on an mbarrier;
//   reduce  every thread reads the P staged vectors at its position, sums them
//           in rank order in binary32, writes the result vector to a shared
//           output tile;
//   gather  the elected thread issues P bulk copies shared -> global, one into
//           every rank's output (the all-gather leaves from on-chip memory; the
//           reduced data never takes a second trip through HBM).
//
// HBM sees long contiguous bursts per stream, and the bytes in flight are set by
// tile size x stages x CTAs, not by how many registers the compiler spends on
// loads.  No multicast of any kind is used.  Synchronisation with the peers is
// the same pair of one-directional signal exchanges as in the register kernel;
// every wait, including the mbarrier waits, is bounded.
#include "symar_device.cuh"
#include "symar_internal.h"

namespace symar {

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return done != 0;
}
// global -> shared of this CTA, completion signalled on `bar` in bytes
__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gsrc, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}
// shared -> global, tracked by the thread's bulk async-group
__device__ __forceinline__ void bulk_store(void *gdst, const void *smem_src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_addr(smem_src)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// at most N groups still READING shared memory
template <int N>
__device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
// every group complete (writes performed)
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// orders this thread's shared-memory writes before later async-proxy reads of them
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }

template <typename E, int P>
__global__ void __launch_bounds__(kMaxThreads) twoshot_bulk_kernel(const KArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    SYMAR_CHECK_BEGIN_ALLREDUCE(a, P);
    const int c = blockIdx.x, r = blockIdx.y, C = gridDim.x;
    const uint32_t t = threadIdx.x, T = blockDim.x;
    const uint32_t S = a.stages, TV = a.tile_vecs, TB = TV * 16u;
    uint64_t *full           = reinterpret_cast<uint64_t *>(smem);          // [S]
    unsigned char *in_tiles  = smem + kBulkBarBytes;                        // [S][P][TB]
    unsigned char *out_tiles = in_tiles + (size_t)S * P * TB;               // [kBulkOutBufs][TB]

    const uint32_t *rcount = reinterpret_cast<const uint32_t *>(counters_near(a, r, c) + kCtrReady);
    const uint32_t *dcount = reinterpret_cast<const uint32_t *>(counters_near(a, r, c) + kCtrDone);

    if (t == 0) {
        for (uint32_t s = 0; s < S; ++s) mbar_init(&full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (a.pdl) pdl_wait();                  // the previous call has left the heap
    uint32_t rwant, dwant;
    bool ok = flag_exchange<P, false>(a, a.ready_off, kPairReady, rcount, r, c, false, true, rwant);
    ok = __syncthreads_and(ok);            // the whole CTA enters the pipeline, or none of it

    // The bulk path moves whole vectors; a partial last vector is done by hand below.
    const uint64_t nv    = a.tail_bytes ? a.nvec - 1 : a.nvec;
    const uint64_t ntile = (nv + TV - 1) / TV;
    const uint64_t mine  = (ntile + P - 1 - r) / P;                          // tiles owned by rank r
    const uint64_t nj    = mine > (uint64_t)c ? (mine - c + C - 1) / C : 0;  // of which this CTA takes
    uint64_t issued = 0;                                                     // tiles whose loads were issued (thread 0)

    // tile i of this CTA -> first vector and vector count
    auto tile_first = [&](uint64_t i) { return (((uint64_t)c + i * C) * P + r) * TV; };
    auto tile_count = [&](uint64_t v0) { return (uint32_t)(nv - v0 < TV ? nv - v0 : TV); };
    auto issue = [&](uint64_t i) {
        const uint32_t s   = (uint32_t)(i % S);
        const uint64_t v0  = tile_first(i);
        const uint32_t nb  = tile_count(v0) * 16u;
        // (checking build: a tile outside the call's input range is not copied, and not waited for)
        uint32_t good = 0;
#pragma unroll
        for (int q = 0; q < P; ++q)
            good += SYMAR_RANGE_OK(a.seg0 + (size_t)q * a.stride + a.in_off + v0 * 16, nb, kRegIn) ? 1u : 0u;
        mbar_expect_tx(&full[s], nb * good);
#pragma unroll
        for (int q = 0; q < P; ++q)
            if (good == (uint32_t)P || SYMAR_RANGE_OK(a.seg0 + (size_t)q * a.stride + a.in_off + v0 * 16, nb, kRegIn))
                bulk_load(in_tiles + ((size_t)s * P + q) * TB, a.seg0 + (size_t)q * a.stride + a.in_off + v0 * 16, nb,
                          &full[s]);
    };

    if (ok && t == 0)
        for (; issued < nj && issued + 1 < S; ++issued) issue(issued);

    uint64_t i = 0;
    for (; ok && i < nj; ++i) {
        const uint32_t s = (uint32_t)(i % S);
        // refill the stage consumed in the previous trip (every thread left it
        // before the barrier that ended that trip)
        if (t == 0 && issued < nj) issue(issued++);
        // wait for this tile: P bulk copies have deposited their bytes
        {
            const uint32_t parity = (uint32_t)((i / S) & 1u);
            Spin spin;
            while (!mbar_try_wait(&full[s], parity)) {
                if (spin.due() && spin.expired(a.spin_ns)) {
                    report_timeout(a.ctl, r, r, c);
                    ok = false;
                    break;
                }
            }
        }
        const uint64_t v0  = tile_first(i);
        const uint32_t nvt = tile_count(v0);
        unsigned char *ot  = out_tiles + (size_t)(i % kBulkOutBufs) * TB;
        if (ok) {
            for (uint32_t k = t; k < nvt; k += T) {
                uint4 x[P];
#pragma unroll
                for (int q = 0; q < P; ++q)
                    x[q] = *reinterpret_cast<const uint4 *>(in_tiles + ((size_t)s * P + q) * TB + (size_t)k * 16);
                *reinterpret_cast<uint4 *>(ot + (size_t)k * 16) = reduce_in_rank_order<E, P>(x);
            }
        }
        fence_proxy_async_smem();
        ok = __syncthreads_and(ok);       // the tile is reduced; or leave together if a wait ran out
        if (!ok) break;
        if (t == 0) {
            // all-gather: the reduced tile leaves shared memory once per rank
#pragma unroll
            for (int q = 0; q < P; ++q)
                if (SYMAR_RANGE_OK(a.seg0 + (size_t)q * a.stride + a.out_off + v0 * 16, nvt * 16u, kRegOut))
                    bulk_store(a.seg0 + (size_t)q * a.stride + a.out_off + v0 * 16, ot, nvt * 16u);
            bulk_commit();
            // The output tile written two trips from now is the one stored in the
            // previous trip: let all but the newest store finish reading.
            bulk_wait_read<1>();
        }
    }
    if (t == 0) {
        bulk_wait_all();          // this CTA's output tiles are in memory
        fence_proxy_async();
        // Only after a wait ran out: loads that were issued but not consumed must
        // land (or be given up on, bounded) before this CTA's shared memory goes away.
        for (uint64_t j = i; !ok && j < issued; ++j) {
            Spin spin;
            while (!mbar_try_wait(&full[j % S], (uint32_t)((j / S) & 1u)))
                if (spin.due() && spin.expired(a.spin_ns)) break;
        }
    }
    // the partial last vector, if any, belongs to the rank that would own its tile
    if (ok && a.tail_bytes != 0 && c == 0 && t == 0 && (int)(((a.nvec - 1) / TV) % P) == r)
        twoshot_vector<E, P>(a, a.nvec - 1);

    __syncthreads();
    flag_exchange<P, true>(a, a.done_off, kPairDone, dcount, r, c, !ok, false, dwant);
    publish_u32(a, r, c, kCtrReady, rwant);
    publish_u32(a, r, c, kCtrDone, dwant);
}

template <typename E>
static KernelFn pick_bulk(int P)
{
    switch (P) {
        case 1: return twoshot_bulk_kernel<E, 1>;
        case 2: return twoshot_bulk_kernel<E, 2>;
        case 4: return twoshot_bulk_kernel<E, 4>;
        case 8: return twoshot_bulk_kernel<E, 8>;
    }
    return nullptr;
}

KernelFn bulk_kernel_for(int dtype, int P)
{
    if (dtype == SYMAR_F32) return pick_bulk<F32>(P);
    if (dtype == SYMAR_BF16) return pick_bulk<BF16>(P);
    return nullptr;
}

}  // namespace symar
